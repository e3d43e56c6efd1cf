// Elementwise kernels that sit between the Monarch passes of the composite calls: the combination step of the
// complex multiply (further down) and the steps of the feed-forward block's backward pass (Section 4: the block
// is trained by the chain rule through a = M1 x + b1, h = GELU(a), y = M2 h + b2).  The two Monarch backward
// passes are the ordinary monarch_bwd kernels; this file holds what sits between them:
//   mlp_act:   h = GELU(a)                                   (a recomputed by a forward pass of M1)
//   mlp_dact:  da = dh * GELU'(a),  db1 += sum_t da,  db2 += sum_t dy
// Both are pure streaming kernels (16-byte accesses, one pass over their operands).
#include "common.cuh"

namespace monarch {
namespace {

constexpr int kThreads = 256;

template <typename T> struct vec16;
template <> struct vec16<float> {
    static constexpr int kElems = 4;
    static __device__ __forceinline__ void load(const float *p, float (&v)[4])
    {
        const float4 q = *reinterpret_cast<const float4 *>(p);
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    }
    static __device__ __forceinline__ void store(float *p, const float (&v)[4])
    {
        *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
};
template <> struct vec16<__nv_bfloat16> {
    static constexpr int kElems = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&v)[8])
    {
        const uint4 q = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, const float (&v)[8])
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t *>(&h2);
        }
        *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// d/da of a/2 (1 + erf(a / sqrt 2)):  Phi(a) + a phi(a)
__device__ __forceinline__ float gelu_erf_grad(float a)
{
    const float cdf = 0.5f * (1.0f + erff(a * 0.70710678118654752440f));
    return cdf + a * 0.39894228040143267794f * expf(-0.5f * a * a);
}

// fp32 tensors get the libm-grade forms; bf16 results are rounded to 8 bits of mantissa, so the cheaper forms
// (error <= 5.1e-5) change nothing there and keep both kernels bound by memory rather than by erff / expf
template <typename T> struct act_math;
template <> struct act_math<float> {
    static __device__ __forceinline__ float gelu(float a) { return gelu_erf(a); }
    static __device__ __forceinline__ float grad(float a) { return gelu_erf_grad(a); }
};
template <> struct act_math<__nv_bfloat16> {
    static __device__ __forceinline__ float gelu(float a) { return gelu_fast(a); }
    static __device__ __forceinline__ float grad(float a) { return gelu_fast_grad(a); }
};

// h[t][q] = GELU(a[t][q] (+ b1[q])); n is a multiple of the vector width
template <typename T>
__global__ void __launch_bounds__(kThreads)
mlp_act_kernel(const T *__restrict__ a, const T *__restrict__ b1, T *__restrict__ h, long long vecs, int n)
{
    constexpr int V = vec16<T>::kElems, U = 4;          // U independent 16-byte loads in flight per thread
    const long long stride = (long long)gridDim.x * kThreads;
    for (long long i0 = (long long)blockIdx.x * kThreads + threadIdx.x; i0 < vecs; i0 += U * stride) {
        float v[U][V];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (i0 + u * stride < vecs) vec16<T>::load(a + (i0 + u * stride) * V, v[u]);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long i = i0 + u * stride;
            if (i >= vecs) break;
            if (b1 != nullptr) {
                float b[V];
                vec16<T>::load(b1 + (int)((i * V) % n), b);
#pragma unroll
                for (int e = 0; e < V; ++e) v[u][e] += b[e];
            }
#pragma unroll
            for (int e = 0; e < V; ++e) v[u][e] = act_math<T>::gelu(v[u][e]);
            vec16<T>::store(h + i * V, v[u]);
        }
    }
}

// One thread owns V consecutive columns and walks a slab of tokens: da = dh * GELU'(a (+ b1)) in place of dh,
// with the column sums of da and dy kept in registers (fp32, from the unrounded da) and added to db1 / db2 once.
template <typename T>
__global__ void __launch_bounds__(kThreads)
mlp_dact_kernel(T *__restrict__ dh, const T *__restrict__ a, const T *__restrict__ b1, const T *__restrict__ dy,
                float *__restrict__ db1, float *__restrict__ db2, long long tokens, int n, int tokens_per_slab)
{
    constexpr int V = vec16<T>::kElems;
    const int col = (blockIdx.x * kThreads + threadIdx.x) * V;
    if (col >= n) return;
    float bias[V], s1[V], s2[V];
#pragma unroll
    for (int e = 0; e < V; ++e) bias[e] = s1[e] = s2[e] = 0.0f;
    if (b1 != nullptr) vec16<T>::load(b1 + col, bias);
    const long long t0 = (long long)blockIdx.y * tokens_per_slab;
    const long long t1 = t0 + tokens_per_slab < tokens ? t0 + tokens_per_slab : tokens;
#pragma unroll 2
    for (long long t = t0; t < t1; ++t) {
        const long long off = t * n + col;
        float g[V], av[V], yv[V];
        vec16<T>::load(dh + off, g);
        vec16<T>::load(a + off, av);
        vec16<T>::load(dy + off, yv);
#pragma unroll
        for (int e = 0; e < V; ++e) {
            g[e] *= act_math<T>::grad(av[e] + bias[e]);
            s1[e] += g[e];
            s2[e] += yv[e];
        }
        vec16<T>::store(dh + off, g);
    }
    if (t1 > t0) {
#pragma unroll
        for (int e = 0; e < V; ++e) {
            atomicAdd(db1 + col + e, s1[e]);
            atomicAdd(db2 + col + e, s2[e]);
        }
    }
}

// Combination step of the complex multiply: with A, B, C, D = M(Lr,Rr), M(Li,Ri), M(Lr,Ri), M(Li,Rr) applied to
// the stacked planes [xr; xi] (each [2][plane] elements),
//   y_re = A[0] - B[0] + sgn (C[1] + D[1]),   y_im = A[1] - B[1] - sgn (C[0] + D[0]),
// sgn = -1 for y = M x and +1 for y = M^H x.
template <typename T>
__global__ void __launch_bounds__(kThreads)
cplx_combine_kernel(const T *__restrict__ A, const T *__restrict__ B, const T *__restrict__ C, const T *__restrict__ D,
                    T *__restrict__ y, long long plane_vecs, float sgn)
{
    constexpr int V = vec16<T>::kElems;
    for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < plane_vecs; i += (long long)gridDim.x * kThreads) {
        float a0[V], a1[V], b0[V], b1[V], c0[V], c1[V], d0[V], d1[V], re[V], im[V];
        const long long o0 = i * V, o1 = (plane_vecs + i) * V;
        vec16<T>::load(A + o0, a0); vec16<T>::load(A + o1, a1);
        vec16<T>::load(B + o0, b0); vec16<T>::load(B + o1, b1);
        vec16<T>::load(C + o0, c0); vec16<T>::load(C + o1, c1);
        vec16<T>::load(D + o0, d0); vec16<T>::load(D + o1, d1);
#pragma unroll
        for (int e = 0; e < V; ++e) {
            re[e] = (a0[e] - b0[e]) + sgn * (c1[e] + d1[e]);
            im[e] = (a1[e] - b1[e]) - sgn * (c0[e] + d0[e]);
        }
        vec16<T>::store(y + o0, re);
        vec16<T>::store(y + o1, im);
    }
}

__global__ void merge_status_kernel(unsigned *outer, unsigned *inner)
{
    const unsigned v = *inner;
    if (v != 0) {
        atomicCAS(outer, 0u, v);
        *inner = 0;
    }
}

template <typename T>
int act_t(const void *a, const void *b1, void *h, int64_t tokens, int n, cudaStream_t s)
{
    const long long vecs = (long long)tokens * n / vec16<T>::kElems;
    if (vecs == 0) return MONARCH_OK;
    long long blocks = (vecs + kThreads - 1) / kThreads;
    if (blocks > 148 * 16) blocks = 148 * 16;
    mlp_act_kernel<T><<<(unsigned)blocks, kThreads, 0, s>>>((const T *)a, (const T *)b1, (T *)h, vecs, n);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

template <typename T>
int dact_t(void *dh, const void *a, const void *b1, const void *dy, float *db1, float *db2, int64_t tokens, int n,
           cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    const int cols_per_block = kThreads * vec16<T>::kElems;
    const int bx = (n + cols_per_block - 1) / cols_per_block;
    // about 16 resident blocks per SM keep enough loads in flight; at least 8 tokens per slab bound the atomics
    long long slabs = (148 * 16 + bx - 1) / bx;
    if (slabs > (tokens + 7) / 8) slabs = (tokens + 7) / 8;
    const int per = (int)((tokens + slabs - 1) / slabs);
    slabs = (tokens + per - 1) / per;
    mlp_dact_kernel<T><<<dim3((unsigned)bx, (unsigned)slabs), kThreads, 0, s>>>((T *)dh, (const T *)a, (const T *)b1,
                                                                               (const T *)dy, db1, db2, tokens, n, per);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

}  // namespace

int mlp_act(const void *a, const void *b1, void *h, int64_t tokens, int n, int dtype, cudaStream_t s)
{
    return dtype == MONARCH_F32 ? act_t<float>(a, b1, h, tokens, n, s) : act_t<__nv_bfloat16>(a, b1, h, tokens, n, s);
}

int mlp_dact(void *dh, const void *a, const void *b1, const void *dy, float *db1, float *db2, int64_t tokens, int n,
             int dtype, cudaStream_t s)
{
    return dtype == MONARCH_F32 ? dact_t<float>(dh, a, b1, dy, db1, db2, tokens, n, s)
                                : dact_t<__nv_bfloat16>(dh, a, b1, dy, db1, db2, tokens, n, s);
}

int cplx_combine(const void *A, const void *B, const void *C, const void *D, void *y, int64_t plane_elems, int adjoint,
                 int dtype, cudaStream_t s)
{
    if (plane_elems == 0) return MONARCH_OK;
    const float sgn = adjoint ? 1.0f : -1.0f;
    const long long vecs = plane_elems / (dtype == MONARCH_F32 ? 4 : 8);
    long long blocks = (vecs + kThreads - 1) / kThreads;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (dtype == MONARCH_F32)
        cplx_combine_kernel<float><<<(unsigned)blocks, kThreads, 0, s>>>((const float *)A, (const float *)B, (const float *)C,
                                                                        (const float *)D, (float *)y, vecs, sgn);
    else
        cplx_combine_kernel<__nv_bfloat16><<<(unsigned)blocks, kThreads, 0, s>>>(
            (const __nv_bfloat16 *)A, (const __nv_bfloat16 *)B, (const __nv_bfloat16 *)C, (const __nv_bfloat16 *)D,
            (__nv_bfloat16 *)y, vecs, sgn);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

int merge_status(unsigned *outer, unsigned *inner, cudaStream_t s)
{
    merge_status_kernel<<<1, 1, 0, s>>>(outer, inner);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

}  // namespace monarch
