// Rectangular Monarch class with wrapped-diagonal blocks (appendix "General Monarch Matrix Parametrization", the
// rectangular definition with b2 != b3):  y = L R x,  R = diag(R_0 .. R_{q-1}) with blocks b2 x b1,  L an r x q grid
// of wrapped-diagonal blocks S_{l,k} of size b3 x b2.  A wrapped diagonal has max(b2, b3) non-zeros: for b2 <= b3 row
// i0 holds one in column i0 mod b2, for b2 > b3 column j0 holds one in row j0 mod b3.  Stored entry e of a block is
// S[i0(e)][j0(e)] with (i0, j0) = (e, e mod b2) or (e mod b3, e); L is stored as Lw[l][k][e].
//
// Every stored entry moves one element of u = R x to one element of y, so when one block size divides the other the
// product is the diagonal-block case with other sizes, and the kernels of that case run on re-labelled weights:
//   b3 = c b2:  rows i0 = a b2 + d of block row l form block row l c + a with diagonal position d:
//               (q, b, r) -> (q, b2, r c),   Lp[d][l c + a][k] = Lw[l][k][a b2 + d]
//   b2 = c b3:  u's blocks of b2 are c blocks of b3, position j0 = a b3 + d is block k c + a, diagonal position d:
//               (q, b, r) -> (q c, b3, r),   Lp[d][l][k c + a] = Lw[l][k][a b3 + d]
// Stage 1 (u = R x) is the diagonal-block stage 1 with b = b2 in both cases.  Otherwise (neither divides the other)
// plain CUDA-core kernels apply the entries where they are.
#include "common.cuh"

namespace monarch {
namespace {

constexpr int kThreads = 256;

__host__ __device__ inline size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }

struct Relabel {
    int r, q, b2, b3, bmax;
    int c;          // ratio of the block sizes
    int up;         // 1: b3 = c b2, 0: b2 = c b3
    int bb, r2, q2; // sizes of the diagonal-block problem
};

Relabel relabel_of(int q, int b2, int b3, int r)
{
    Relabel m;
    m.r = r; m.q = q; m.b2 = b2; m.b3 = b3; m.bmax = b2 > b3 ? b2 : b3;
    m.up = b3 % b2 == 0;
    m.c = m.up ? b3 / b2 : b2 / b3;
    m.bb = m.up ? b2 : b3;
    m.r2 = m.up ? r * m.c : r;
    m.q2 = m.up ? q : q * m.c;
    return m;
}

// index of stored entry (l, k, e) in the diagonal-block layout Lp[bb][r2][q2]
__device__ __forceinline__ size_t relabelled(const Relabel &m, int l, int k, int e)
{
    const int a = e / m.bb, d = e % m.bb;
    return m.up ? ((size_t)d * m.r2 + (l * m.c + a)) * m.q2 + k : ((size_t)d * m.r2 + l) * m.q2 + (k * m.c + a);
}

template <typename T>
__global__ void relabel_kernel(const T *__restrict__ Lw, T *__restrict__ Lp, const Relabel m)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x, total = (size_t)m.r * m.q * m.bmax;
    if (idx >= total) return;
    const int e = (int)(idx % m.bmax), k = (int)((idx / m.bmax) % m.q), l = (int)(idx / ((size_t)m.bmax * m.q));
    Lp[relabelled(m, l, k, e)] = Lw[idx];
}

// dLw = (accumulate ? dLw : 0) + dLp re-labelled back
__global__ void relabel_back_kernel(const float *__restrict__ dLp, float *__restrict__ dLw, const Relabel m, int accumulate)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x, total = (size_t)m.r * m.q * m.bmax;
    if (idx >= total) return;
    const int e = (int)(idx % m.bmax), k = (int)((idx / m.bmax) % m.q), l = (int)(idx / ((size_t)m.bmax * m.q));
    const float v = dLp[relabelled(m, l, k, e)];
    dLw[idx] = accumulate ? dLw[idx] + v : v;
}

// ---- general sizes: the entries applied where they are --------------------------------------------------------------
// y[t][l*b3 + i0] = sum_k sum_{e: i0(e) = i0} Lw[l][k][e] u[t][k*b2 + j0(e)]
template <typename T>
__global__ void stage2_kernel(const T *__restrict__ u, const T *__restrict__ Lw, T *__restrict__ y, long long tokens, int q,
                              int b2, int b3, int r)
{
    const int bmax = b2 > b3 ? b2 : b3, n2 = q * b2, n3 = r * b3;
    const long long total = tokens * n3;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
        const long long t = idx / n3;
        const int o = (int)(idx % n3), l = o / b3, i0 = o % b3;
        const T *ut = u + t * n2, *w = Lw + (size_t)l * q * bmax;
        float acc = 0.f;
        if (b2 <= b3) {
            const int j0 = i0 % b2;
            for (int k = 0; k < q; ++k) acc = fmaf(elem<T>::load(w + (size_t)k * bmax + i0), elem<T>::load(ut + k * b2 + j0), acc);
        } else {
            for (int e = i0; e < b2; e += b3)
                for (int k = 0; k < q; ++k) acc = fmaf(elem<T>::load(w + (size_t)k * bmax + e), elem<T>::load(ut + k * b2 + e), acc);
        }
        elem<T>::store(y + idx, acc);
    }
}

// du[t][k*b2 + j0] = sum_l sum_{e: j0(e) = j0} Lw[l][k][e] dy[t][l*b3 + i0(e)]
template <typename T>
__global__ void stage2_adjoint_kernel(const T *__restrict__ dy, const T *__restrict__ Lw, T *__restrict__ du, long long tokens,
                                      int q, int b2, int b3, int r)
{
    const int bmax = b2 > b3 ? b2 : b3, n2 = q * b2, n3 = r * b3;
    const long long total = tokens * n2;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
        const long long t = idx / n2;
        const int pcol = (int)(idx % n2), k = pcol / b2, j0 = pcol % b2;
        const T *dt = dy + t * n3;
        float acc = 0.f;
        if (b2 <= b3) {
            for (int e = j0; e < b3; e += b2)
                for (int l = 0; l < r; ++l)
                    acc = fmaf(elem<T>::load(Lw + ((size_t)l * q + k) * bmax + e), elem<T>::load(dt + l * b3 + e), acc);
        } else {
            const int i0 = j0 % b3;
            for (int l = 0; l < r; ++l)
                acc = fmaf(elem<T>::load(Lw + ((size_t)l * q + k) * bmax + j0), elem<T>::load(dt + l * b3 + i0), acc);
        }
        elem<T>::store(du + idx, acc);
    }
}

// dLw[l][k][e] += sum over a slab of tokens of dy[t][l*b3 + i0(e)] u[t][k*b2 + j0(e)]   (blockIdx.y = slab)
template <typename T>
__global__ void dL_kernel(const T *__restrict__ dy, const T *__restrict__ u, float *__restrict__ dLw, long long tokens, int slab,
                          int q, int b2, int b3, int r)
{
    const int bmax = b2 > b3 ? b2 : b3, n2 = q * b2, n3 = r * b3;
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x, total = (size_t)r * q * bmax;
    if (idx >= total) return;
    const int e = (int)(idx % bmax), k = (int)((idx / bmax) % q), l = (int)(idx / ((size_t)bmax * q));
    const int i0 = b2 <= b3 ? e : e % b3, j0 = b2 <= b3 ? e % b2 : e;
    const long long t0 = (long long)blockIdx.y * slab, t1 = t0 + slab < tokens ? t0 + slab : tokens;
    float acc = 0.f;
    for (long long t = t0; t < t1; ++t)
        acc = fmaf(elem<T>::load(dy + t * n3 + l * b3 + i0), elem<T>::load(u + t * n2 + k * b2 + j0), acc);
    atomicAdd(dLw + idx, acc);
}

int grid_for(long long total)
{
    long long g = (total + kThreads - 1) / kThreads;
    if (g > 148 * 32) g = 148 * 32;
    return g < 1 ? 1 : (int)g;
}

bool divisible(int b2, int b3) { return b3 % b2 == 0 || b2 % b3 == 0; }

int stage1(const void *x, const void *R, void *u, int64_t tokens, int q, int b1, int b2, int dtype, bool fast, unsigned *status,
           cudaStream_t s)
{
    if (fast && rect_stage1_tc_available(q, b1, b2, dtype)) return rect_stage1_tc(x, R, u, tokens, q, b1, b2, status, s);
    return rect_stage1_simt(x, R, u, tokens, q, b1, b2, dtype, 0, s);
}

// stage 2 of the diagonal-block case (wt = 1: its adjoint, with the roles of q and r exchanged by the caller)
int stage2_diag(const void *in, const void *Lp, void *out, int64_t tokens, int q, int b, int r, int dtype, int wt, bool fast,
                unsigned *status, cudaStream_t s)
{
    if (fast && rect_stage2_stream_available(q, b, r, dtype)) return rect_stage2_stream(in, Lp, out, tokens, q, b, r, wt, status, s);
    return rect_stage2_simt(in, Lp, out, tokens, q, b, r, dtype, wt, s);
}

}  // namespace

// Workspaces: forward [status][u][Lp]; backward [status][u][du][Lp][dLp (fp32)]
size_t rectw_workspace_bytes(int64_t tokens, int q, int b2, int b3, int r, int dtype)
{
    const size_t es = dtype == MONARCH_F32 ? 4 : 2, bmax = b2 > b3 ? b2 : b3;
    return rect_workspace_bytes(tokens, q, b2, dtype) + round256((size_t)r * q * bmax * es);
}
size_t rectw_bwd_workspace_bytes(int64_t tokens, int q, int b2, int b3, int r, int dtype)
{
    const size_t es = dtype == MONARCH_F32 ? 4 : 2, bmax = b2 > b3 ? b2 : b3;
    return MONARCH_STATUS_BYTES + 2 * round256((size_t)tokens * q * b2 * es) + round256((size_t)r * q * bmax * es) +
           round256((size_t)r * q * bmax * sizeof(float));
}

int rectw_fwd(const void *x, const void *Lw, const void *R, void *y, int64_t tokens, int q, int b1, int b2, int b3, int r,
              int dtype, bool fast, void *ws, cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    const size_t es = dtype == MONARCH_F32 ? 4 : 2;
    unsigned *status = (unsigned *)ws;
    char *u = (char *)ws + MONARCH_STATUS_BYTES;
    char *Lp = u + round256((size_t)tokens * q * b2 * es);
    MONARCH_TRY(stage1(x, R, u, tokens, q, b1, b2, dtype, fast, status, s));
    if (divisible(b2, b3)) {
        const Relabel m = relabel_of(q, b2, b3, r);
        const int g = grid_for((long long)r * q * m.bmax);
        if (dtype == MONARCH_F32) relabel_kernel<float><<<g, kThreads, 0, s>>>((const float *)Lw, (float *)Lp, m);
        else relabel_kernel<__nv_bfloat16><<<g, kThreads, 0, s>>>((const __nv_bfloat16 *)Lw, (__nv_bfloat16 *)Lp, m);
        note_launch();
        MONARCH_CUDA_TRY(cudaGetLastError());
        return stage2_diag(u, Lp, y, tokens, m.q2, m.bb, m.r2, dtype, 0, fast, status, s);
    }
    const int g = grid_for(tokens * r * b3);
    if (dtype == MONARCH_F32)
        stage2_kernel<float><<<g, kThreads, 0, s>>>((const float *)u, (const float *)Lw, (float *)y, tokens, q, b2, b3, r);
    else
        stage2_kernel<__nv_bfloat16><<<g, kThreads, 0, s>>>((const __nv_bfloat16 *)u, (const __nv_bfloat16 *)Lw, (__nv_bfloat16 *)y,
                                                           tokens, q, b2, b3, r);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

int rectw_bwd(const void *x, const void *dy, const void *Lw, const void *R, void *dx, float *dLw, float *dR, int accumulate,
              int64_t tokens, int q, int b1, int b2, int b3, int r, int dtype, bool fast, void *ws, cudaStream_t s)
{
    const size_t es = dtype == MONARCH_F32 ? 4 : 2, bmax = b2 > b3 ? b2 : b3;
    const size_t lw = (size_t)r * q * bmax, rb = (size_t)q * b2 * b1;
    if (!accumulate) {
        MONARCH_CUDA_TRY(cudaMemsetAsync(dLw, 0, lw * sizeof(float), s));
        MONARCH_CUDA_TRY(cudaMemsetAsync(dR, 0, rb * sizeof(float), s));
    }
    if (tokens == 0) return MONARCH_OK;
    unsigned *status = (unsigned *)ws;
    char *u = (char *)ws + MONARCH_STATUS_BYTES;
    char *du = u + round256((size_t)tokens * q * b2 * es);
    char *Lp = du + round256((size_t)tokens * q * b2 * es);
    float *dLp = (float *)(Lp + round256(lw * es));
    MONARCH_TRY(stage1(x, R, u, tokens, q, b1, b2, dtype, fast, status, s));
    const bool div = divisible(b2, b3);
    const Relabel m = relabel_of(q, b2, b3, r);
    if (div) {
        const int g = grid_for((long long)lw);
        if (dtype == MONARCH_F32) relabel_kernel<float><<<g, kThreads, 0, s>>>((const float *)Lw, (float *)Lp, m);
        else relabel_kernel<__nv_bfloat16><<<g, kThreads, 0, s>>>((const __nv_bfloat16 *)Lw, (__nv_bfloat16 *)Lp, m);
        note_launch();
        MONARCH_CUDA_TRY(cudaGetLastError());
        // du = L^T dy: stage 2 with the roles of q and r exchanged and the blocks read transposed
        MONARCH_TRY(stage2_diag(dy, Lp, du, tokens, m.r2, m.bb, m.q2, dtype, 1, fast, status, s));
    } else {
        const int g = grid_for(tokens * q * b2);
        if (dtype == MONARCH_F32)
            stage2_adjoint_kernel<float><<<g, kThreads, 0, s>>>((const float *)dy, (const float *)Lw, (float *)du, tokens, q, b2, b3, r);
        else
            stage2_adjoint_kernel<__nv_bfloat16><<<g, kThreads, 0, s>>>((const __nv_bfloat16 *)dy, (const __nv_bfloat16 *)Lw,
                                                                       (__nv_bfloat16 *)du, tokens, q, b2, b3, r);
        note_launch();
        MONARCH_CUDA_TRY(cudaGetLastError());
    }
    // dx = blockdiag(R)^T du and dR: the diagonal-block case with b = b2
    if (fast && rect_stage1_tc_available(q, b1, b2, dtype))
        MONARCH_TRY(rect_stage1_adjoint_tc(du, R, dx, tokens, q, b1, b2, status, s));
    else
        MONARCH_TRY(rect_stage1_simt(du, R, dx, tokens, q, b2, b1, dtype, 1, s));
    const bool tc_dR = fast && rect_wgrad_R_tc_available(q, b1, b2, dtype);
    if (tc_dR) MONARCH_TRY(rect_wgrad_R_tc(du, x, dR, tokens, q, b1, b2, status, s));
    else MONARCH_TRY(rect_wgrad_simt(x, dy, u, du, nullptr, dR, tokens, q, b1, b2, 1, dtype, 0, 1, s));
    if (div) {
        // dLp of the re-labelled problem (into zeroed scratch), then back into the caller's layout
        MONARCH_CUDA_TRY(cudaMemsetAsync(dLp, 0, lw * sizeof(float), s));
        const bool stream_dL = fast && rect_stage2_stream_available(m.q2, m.bb, m.r2, dtype);
        if (stream_dL) MONARCH_TRY(rect_dl_stream(dy, u, dLp, tokens, m.q2, m.bb, m.r2, status, s));
        else MONARCH_TRY(rect_wgrad_simt(x, dy, u, du, dLp, nullptr, tokens, m.q2, 1, m.bb, m.r2, dtype, 1, 0, s));
        relabel_back_kernel<<<grid_for((long long)lw), kThreads, 0, s>>>(dLp, dLw, m, 1);
        note_launch();
        MONARCH_CUDA_TRY(cudaGetLastError());
        return MONARCH_OK;
    }
    const int slab = 256;
    const dim3 grid((unsigned)((lw + kThreads - 1) / kThreads), (unsigned)((tokens + slab - 1) / slab));
    if (grid.y > 65535) return MONARCH_ERR_UNSUPPORTED;
    if (dtype == MONARCH_F32)
        dL_kernel<float><<<grid, kThreads, 0, s>>>((const float *)dy, (const float *)u, dLw, tokens, slab, q, b2, b3, r);
    else
        dL_kernel<__nv_bfloat16><<<grid, kThreads, 0, s>>>((const __nv_bfloat16 *)dy, (const __nv_bfloat16 *)u, dLw, tokens, slab, q,
                                                          b2, b3, r);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

}  // namespace monarch
