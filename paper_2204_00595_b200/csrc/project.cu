// Conversions between a dense n x n matrix and the Monarch factors (n = m*m):
//   monarch_dense    Eq. (2):       M[l*m+j][k*m+i] = L[j][l][k] R[k][j][i]
//   monarch_project  Algorithm 1:   view A as A~[l][j][k][i] = A[l*m+j][k*m+i]; for every (j, k) replace the m x m
//                                   slice A~[:, j, k, :] by its best rank-1 approximation sigma u v^T and store
//                                   L[j][:, k] = sqrt(sigma) u,  R[k][j][:] = sqrt(sigma) v.
// The m*m slices are independent: one CTA per slice.  The leading singular triplet comes from a one-sided Jacobi
// iteration in shared memory (columns are rotated in pairs until they are mutually orthogonal; their norms are then
// the singular values and the normalised columns the left singular vectors), which converges at the same rate
// whatever the gap between the first two singular values - a power iteration would not.  v = S^T u / sigma is one
// more pass over the slice.  Arithmetic is fp32 whatever the storage dtype.
#include "common.cuh"

namespace monarch {
namespace {

template <typename T>
__global__ void __launch_bounds__(256)
dense_kernel(const T *__restrict__ L, const T *__restrict__ R, T *__restrict__ M, int m)
{
    // one CTA per output row (l, j); thread -> column k*m + i
    const int row = blockIdx.x, l = row / m, j = row % m, n = m * m;
    for (int col = threadIdx.x; col < n; col += 256) {
        const int k = col / m, i = col % m;
        const float v = elem<T>::load(L + ((size_t)j * m + l) * m + k) * elem<T>::load(R + ((size_t)k * m + j) * m + i);
        elem<T>::store(M + (size_t)row * n + col, v);
    }
}

constexpr int kMaxSweeps = 30;
// columns count as orthogonal below this cosine: a few times the rounding noise of an fp32 dot product of m terms
constexpr float kOrthoTol = 2e-6f;

// Rotation counter for the benchmark's FLOP count (optional, may be null).
// A column pair is handled by G lanes (m/G rows each): G = 8 for m <= 64, so that a warp rotates four pairs at once
// - with 64-element columns a whole warp per pair would spend most of its instructions on shuffle and scalar work
// replicated over 32 lanes - and G = 32 for m = 128, where the strided rows of four different columns would
// collide in the shared-memory banks.  Several CTAs share an SM.
template <int M> struct ProjectCfg {
    static constexpr int kG = M >= 128 ? 32 : 8;
    static constexpr int kPairsPerPass = 32 / kG;                       // pairs a warp rotates at once
    static constexpr int kWarps = M >= 128 ? 32 : (M / 8 < 2 ? 2 : M / 8);
    static constexpr int kPasses = (M / 2) / (kWarps * kPairsPerPass);  // passes per round
};

template <typename T, int M>
__global__ void __launch_bounds__(ProjectCfg<M>::kWarps * 32)
project_kernel(const T *__restrict__ A, T *__restrict__ L, T *__restrict__ R, unsigned long long *rotations)
{
    using C = ProjectCfg<M>;
    constexpr int N = M * M;
    constexpr int kWarps = C::kWarps, G = C::kG;
    static_assert(kWarps * C::kPairsPerPass * C::kPasses == M / 2, "a round covers every column once");
    constexpr int kPitch = M + 1;                         // column pitch in floats (odd: no bank conflicts)
    constexpr int kRows = M / G;                          // rows per lane
    extern __shared__ float cols[];                       // cols[i * kPitch + l] = S[l][i]
    __shared__ float red_val[32];
    __shared__ int red_idx[32];
    __shared__ float u_s[M];
    __shared__ float sigma_s;
    __shared__ int best_s;

    const int j = blockIdx.x / M, k = blockIdx.x % M;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = lane / G, sub = lane % G;
    const T *slice = A + (size_t)j * N + (size_t)k * M;   // element (l, i) at slice[l * M * N + i]

    for (int e = threadIdx.x; e < M * M; e += kWarps * 32) {
        const int l = e / M, i = e % M;
        cols[i * kPitch + l] = elem<T>::load(slice + (size_t)l * M * N + i);
    }
    __syncthreads();

    unsigned my_rot = 0;
    for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
        int rotated = 0;
        for (int rr = 0; rr < M - 1; ++rr) {
#pragma unroll
            for (int pass = 0; pass < C::kPasses; ++pass) {
                // round-robin tournament: column M-1 stays, the others move round a circle of M-1 seats
                const int p = (warp * C::kPasses + pass) * C::kPairsPerPass + grp;
                int ca = rr + p, cb = rr - p + (M - 1);
                if (ca >= M - 1) ca -= M - 1;
                if (cb >= M - 1) cb -= M - 1;
                if (p == 0) ca = M - 1;
                float *a = cols + ca * kPitch + sub, *b = cols + cb * kPitch + sub;
                float av[kRows], bv[kRows];
                float aa = 0.0f, bb = 0.0f, ab = 0.0f;
#pragma unroll
                for (int q = 0; q < kRows; ++q) {
                    av[q] = a[G * q];
                    bv[q] = b[G * q];
                    aa = fmaf(av[q], av[q], aa);
                    bb = fmaf(bv[q], bv[q], bb);
                    ab = fmaf(av[q], bv[q], ab);
                }
#pragma unroll
                for (int o = G / 2; o > 0; o >>= 1) {
                    aa += __shfl_xor_sync(0xffffffffu, aa, o);
                    bb += __shfl_xor_sync(0xffffffffu, bb, o);
                    ab += __shfl_xor_sync(0xffffffffu, ab, o);
                }
                // rotate unless the two columns are already orthogonal to working precision.  The angle only has to
                // be roughly right (orthogonality is re-tested every sweep, and the factors are formed from a
                // re-normalised column), so the fast reciprocal / square-root forms are enough.
                if (ab * ab > (kOrthoTol * kOrthoTol) * (aa * bb)) {
                    // clamped: columns that are pure rounding noise (rank-deficient slices) give huge ratios
                    const float zeta = fmaxf(fminf(__fdividef(bb - aa, 2.0f * ab), 1e15f), -1e15f);
                    const float w = fmaf(zeta, zeta, 1.0f);
                    const float t = copysignf(__fdividef(1.0f, fabsf(zeta) + w * rsqrtf(w)), zeta);
                    const float c = rsqrtf(fmaf(t, t, 1.0f)), s = c * t;
#pragma unroll
                    for (int q = 0; q < kRows; ++q) {
                        a[G * q] = c * av[q] - s * bv[q];
                        b[G * q] = s * av[q] + c * bv[q];
                    }
                    rotated = 1;
                    if (sub == 0) ++my_rot;
                }
            }
            __syncthreads();
        }
        if (!__syncthreads_or(rotated)) break;
    }
    if (rotations != nullptr && my_rot) atomicAdd(rotations, (unsigned long long)my_rot);

    // the column of largest norm carries sigma_1 u_1
    float best = -1.0f;
    int best_i = 0;
    for (int i = threadIdx.x; i < M; i += kWarps * 32) {
        float s2 = 0.0f;
        for (int l = 0; l < M; ++l) s2 = fmaf(cols[i * kPitch + l], cols[i * kPitch + l], s2);
        if (s2 > best) { best = s2; best_i = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
        if (ov > best || (ov == best && oi < best_i)) { best = ov; best_i = oi; }
    }
    if (lane == 0) { red_val[warp] = best; red_idx[warp] = best_i; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float bv = red_val[0];
        int bi = red_idx[0];
        for (int w = 1; w < kWarps; ++w)
            if (red_val[w] > bv || (red_val[w] == bv && red_idx[w] < bi)) { bv = red_val[w]; bi = red_idx[w]; }
        sigma_s = sqrtf(fmaxf(bv, 0.0f));
        best_s = bi;
    }
    __syncthreads();
    const float sigma = sigma_s, root = sqrtf(sigma);
    const float inv = sigma > 0.0f ? 1.0f / sigma : 0.0f;
    for (int l = threadIdx.x; l < M; l += kWarps * 32) {
        const float ul = cols[best_s * kPitch + l] * inv;
        u_s[l] = ul;
        elem<T>::store(L + ((size_t)j * M + l) * M + k, root * ul);
    }
    __syncthreads();
    // v = S^T u / sigma from the original slice (the shared copy has been rotated), scaled by sqrt(sigma)
    for (int i = threadIdx.x; i < M; i += kWarps * 32) {
        float acc = 0.0f;
        for (int l = 0; l < M; ++l) acc = fmaf(elem<T>::load(slice + (size_t)l * M * N + i), u_s[l], acc);
        elem<T>::store(R + ((size_t)k * M + j) * M + i, root * acc * inv);
    }
}

template <typename T, int M>
int launch_project(const void *A, void *L, void *R, unsigned long long *rotations, cudaStream_t s)
{
    constexpr int kWarps = ProjectCfg<M>::kWarps;
    constexpr int smem = M * (M + 1) * (int)sizeof(float);
    static bool attr = false;
    if (!attr && smem > 48 * 1024) {
        MONARCH_CUDA_TRY(cudaFuncSetAttribute(project_kernel<T, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attr = true;
    }
    project_kernel<T, M><<<M * M, kWarps * 32, smem, s>>>((const T *)A, (T *)L, (T *)R, rotations);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

template <typename T>
int project_t(const void *A, void *L, void *R, int m, unsigned long long *rotations, cudaStream_t s)
{
    switch (m) {
        case 16:  return launch_project<T, 16>(A, L, R, rotations, s);
        case 32:  return launch_project<T, 32>(A, L, R, rotations, s);
        case 64:  return launch_project<T, 64>(A, L, R, rotations, s);
        case 128: return launch_project<T, 128>(A, L, R, rotations, s);
    }
    return MONARCH_ERR_UNSUPPORTED;
}

}  // namespace

int dense_from_factors(const void *L, const void *R, void *M, int m, int dtype, cudaStream_t s)
{
    if (dtype == MONARCH_F32)
        dense_kernel<float><<<m * m, 256, 0, s>>>((const float *)L, (const float *)R, (float *)M, m);
    else
        dense_kernel<__nv_bfloat16><<<m * m, 256, 0, s>>>((const __nv_bfloat16 *)L, (const __nv_bfloat16 *)R,
                                                          (__nv_bfloat16 *)M, m);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

int project_to_factors(const void *A, void *L, void *R, int m, int dtype, unsigned long long *rotations, cudaStream_t s)
{
    return dtype == MONARCH_F32 ? project_t<float>(A, L, R, m, rotations, s)
                                : project_t<__nv_bfloat16>(A, L, R, m, rotations, s);
}

}  // namespace monarch
