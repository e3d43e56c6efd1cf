// Staged kernel family: one block-diagonal stage per launch on the CUDA cores (FFMA).
//
// The Monarch product factors as  M = (P L)(P R)  because P = P^T (Section 3.1), so the
// forward pass is the same operation applied twice: multiply every length-m segment of the
// input by its block, then scatter the result with the stride permutation.  The adjoint
// M^T = (R^T P)(L^T P) is the mirrored operation (gather with P, multiply by the transposed
// block).  The weight gradients are token-contracted outer products of a stage's input and
// the adjoint of its output.  The intermediate (u or du) lives in caller-provided workspace.
//
// This family serves float32 (where tensor cores cannot meet the 1e-5 tolerance) and every
// size that has no fused tensor-core kernel.  It is arithmetic-bound, not HBM-bound.
#include <mutex>

#include "common.cuh"

namespace monarch {
namespace {

constexpr int kThreads = 256;
constexpr int kTokTile = 64;   // tokens per CTA in a stage
constexpr int kWgChunk = 32;   // tokens per shared-memory chunk in the weight-gradient kernel

struct Strides {          // element (blk, e) of a token row sits at blk*sb + e*se
    long long sb, se;
};

// out[t][(b, e)] = act( sum_c W(b; e, c) * in[t][(b, c)] + bias[(b, e)] )
// ADJ == false: W(b; e, c) = W[b][e][c]  (multiply by the block)
// ADJ == true : W(b; e, c) = W[b][c][e]  (multiply by the transposed block)
template <typename T, int M, bool ADJ>
__global__ void __launch_bounds__(kThreads)
stage_kernel(const T *__restrict__ in, const T *__restrict__ W, T *__restrict__ out,
             const T *__restrict__ bias, int gelu, long long tokens, Strides is, Strides os)
{
    extern __shared__ float smem[];
    float *Ws = smem;                        // [M][M+1]: Ws[c][e]
    float *xs = smem + M * (M + 1);          // [kTokTile][M]
    constexpr int n = M * M;
    const int b = blockIdx.y;
    const long long t0 = (long long)blockIdx.x * kTokTile;
    const int tid = threadIdx.x;

    const T *Wb = W + (size_t)b * M * M;
    for (int q = tid; q < M * M; q += kThreads) {
        const int r = q / M, c = q % M;      // Wb[r][c], coalesced over c
        const float w = elem<T>::load(Wb + q);
        if (ADJ) Ws[r * (M + 1) + c] = w;    // contraction index is the row
        else     Ws[c * (M + 1) + r] = w;    // contraction index is the column
    }
    for (int q = tid; q < kTokTile * M; q += kThreads) {
        const int tt = q / M, c = q % M;
        const long long t = t0 + tt;
        xs[q] = (t < tokens) ? elem<T>::load(in + (size_t)t * n + b * is.sb + c * is.se) : 0.0f;
    }
    __syncthreads();

    constexpr int RE = M / 16;               // outputs per thread
    constexpr int RT = kTokTile / 16;        // tokens per thread
    const int tx = tid & 15, ty = tid >> 4;
    float acc[RT][RE];
#pragma unroll
    for (int q = 0; q < RT; ++q)
#pragma unroll
        for (int r = 0; r < RE; ++r) acc[q][r] = 0.0f;

    for (int c = 0; c < M; ++c) {
        float w[RE], a[RT];
#pragma unroll
        for (int r = 0; r < RE; ++r) w[r] = Ws[c * (M + 1) + tx + 16 * r];
#pragma unroll
        for (int q = 0; q < RT; ++q) a[q] = xs[(ty + 16 * q) * M + c];
#pragma unroll
        for (int q = 0; q < RT; ++q)
#pragma unroll
            for (int r = 0; r < RE; ++r) acc[q][r] = fmaf(a[q], w[r], acc[q][r]);
    }

#pragma unroll
    for (int q = 0; q < RT; ++q) {
        const long long t = t0 + ty + 16 * q;
        if (t >= tokens) continue;
#pragma unroll
        for (int r = 0; r < RE; ++r) {
            const int e = tx + 16 * r;
            const long long col = b * os.sb + e * os.se;
            float v = acc[q][r];
            if (bias) v += elem<T>::load(bias + col);
            if (gelu) v = gelu_erf(v);
            elem<T>::store(out + (size_t)t * n + col, v);
        }
    }
}

// part[slab][b][p][q] = sum_{t in slab} A[t][(b, p)] * B[t][b*M + q]
template <typename T, int M>
__global__ void __launch_bounds__(kThreads)
wgrad_kernel(const T *__restrict__ A, Strides as, const T *__restrict__ B,
             float *__restrict__ part, long long tokens, long long slab_tokens)
{
    __shared__ float As[kWgChunk][M];
    __shared__ float Bs[kWgChunk][M];
    constexpr int n = M * M;
    constexpr int RE = M / 16;
    const int b = blockIdx.x;
    const int slab = blockIdx.y;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    long long t_begin = (long long)slab * slab_tokens;
    long long t_end = t_begin + slab_tokens;
    if (t_end > tokens) t_end = tokens;

    float acc[RE][RE];
#pragma unroll
    for (int r = 0; r < RE; ++r)
#pragma unroll
        for (int c = 0; c < RE; ++c) acc[r][c] = 0.0f;

    for (long long tc = t_begin; tc < t_end; tc += kWgChunk) {
        for (int q = tid; q < kWgChunk * M; q += kThreads) {
            const int tt = q / M, e = q % M;
            const long long t = tc + tt;
            const bool ok = t < t_end;
            As[tt][e] = ok ? elem<T>::load(A + (size_t)t * n + b * as.sb + e * as.se) : 0.0f;
            Bs[tt][e] = ok ? elem<T>::load(B + (size_t)t * n + b * M + e) : 0.0f;
        }
        __syncthreads();
#pragma unroll 4
        for (int tt = 0; tt < kWgChunk; ++tt) {
            float a[RE], bb[RE];
#pragma unroll
            for (int r = 0; r < RE; ++r) a[r] = As[tt][ty + 16 * r];
#pragma unroll
            for (int c = 0; c < RE; ++c) bb[c] = Bs[tt][tx + 16 * c];
#pragma unroll
            for (int r = 0; r < RE; ++r)
#pragma unroll
                for (int c = 0; c < RE; ++c) acc[r][c] = fmaf(a[r], bb[c], acc[r][c]);
        }
        __syncthreads();
    }
    float *dst = part + ((size_t)slab * M + b) * M * M;
#pragma unroll
    for (int r = 0; r < RE; ++r)
#pragma unroll
        for (int c = 0; c < RE; ++c) dst[(ty + 16 * r) * M + tx + 16 * c] = acc[r][c];
}

// out[e] = (accumulate ? out[e] : 0) + sum_s part[s][e], slabs added in index order.
__global__ void reduce_slabs_kernel(const float *__restrict__ part, float *__restrict__ out,
                                    long long elems, int slabs, int accumulate)
{
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= elems) return;
    float s = accumulate ? out[e] : 0.0f;
    for (int k = 0; k < slabs; ++k) s += part[(size_t)k * elems + e];
    out[e] = s;
}

template <typename T, int M, bool ADJ>
int launch_stage(const void *in, const void *W, void *out, const void *bias, int gelu,
                 int64_t tokens, Strides is, Strides os, cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    const size_t smem = (size_t)(M * (M + 1) + kTokTile * M) * sizeof(float);
    auto kern = stage_kernel<T, M, ADJ>;
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid((unsigned)((tokens + kTokTile - 1) / kTokTile), M);
    kern<<<grid, kThreads, smem, s>>>((const T *)in, (const T *)W, (T *)out, (const T *)bias, gelu,
                                      tokens, is, os);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

template <typename T, bool ADJ>
int stage_m(int m, const void *in, const void *W, void *out, const void *bias, int gelu,
            int64_t tokens, cudaStream_t s)
{
    // multiply-then-permute (ADJ=false) reads natural order and writes with stride m;
    // permute-then-multiply (ADJ=true) reads with stride m and writes natural order.
    const Strides nat = {m, 1}, perm = {1, m};
    const Strides is = ADJ ? perm : nat, os = ADJ ? nat : perm;
    switch (m) {
        case 16:  return launch_stage<T, 16, ADJ>(in, W, out, bias, gelu, tokens, is, os, s);
        case 32:  return launch_stage<T, 32, ADJ>(in, W, out, bias, gelu, tokens, is, os, s);
        case 64:  return launch_stage<T, 64, ADJ>(in, W, out, bias, gelu, tokens, is, os, s);
        case 128: return launch_stage<T, 128, ADJ>(in, W, out, bias, gelu, tokens, is, os, s);
    }
    return MONARCH_ERR_UNSUPPORTED;
}

int stage(int dtype, bool adj, int m, const void *in, const void *W, void *out, const void *bias,
          int gelu, int64_t tokens, cudaStream_t s)
{
    if (dtype == MONARCH_F32)
        return adj ? stage_m<float, true>(m, in, W, out, bias, gelu, tokens, s)
                   : stage_m<float, false>(m, in, W, out, bias, gelu, tokens, s);
    if (dtype == MONARCH_BF16)
        return adj ? stage_m<__nv_bfloat16, true>(m, in, W, out, bias, gelu, tokens, s)
                   : stage_m<__nv_bfloat16, false>(m, in, W, out, bias, gelu, tokens, s);
    return MONARCH_ERR_UNSUPPORTED;
}

int wgrad_slabs(int64_t tokens, int m)
{
    // enough CTAs to fill the machine a few times over, at least 256 tokens per slab
    long long by_grid = (4 * 148 + m - 1) / m;
    long long by_tokens = (tokens + 255) / 256;
    long long s = by_grid < by_tokens ? by_grid : by_tokens;
    return (int)(s < 1 ? 1 : s);
}

template <typename T, int M>
int launch_wgrad(const void *A, Strides as, const void *B, float *part, int64_t tokens, int slabs,
                 cudaStream_t s)
{
    const long long slab_tokens = (tokens + slabs - 1) / slabs;
    dim3 grid(M, slabs);
    wgrad_kernel<T, M><<<grid, kThreads, 0, s>>>((const T *)A, as, (const T *)B, part, tokens,
                                                 slab_tokens);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

template <typename T>
int wgrad_m(int m, const void *A, Strides as, const void *B, float *part, int64_t tokens,
            int slabs, cudaStream_t s)
{
    switch (m) {
        case 16:  return launch_wgrad<T, 16>(A, as, B, part, tokens, slabs, s);
        case 32:  return launch_wgrad<T, 32>(A, as, B, part, tokens, slabs, s);
        case 64:  return launch_wgrad<T, 64>(A, as, B, part, tokens, slabs, s);
        case 128: return launch_wgrad<T, 128>(A, as, B, part, tokens, slabs, s);
    }
    return MONARCH_ERR_UNSUPPORTED;
}

int wgrad(int dtype, int m, const void *A, Strides as, const void *B, float *part, float *out,
          int accumulate, int64_t tokens, cudaStream_t s)
{
    const long long elems = (long long)m * m * m;
    if (tokens == 0) {
        if (!accumulate) MONARCH_CUDA_TRY(cudaMemsetAsync(out, 0, elems * sizeof(float), s));
        return MONARCH_OK;
    }
    const int slabs = wgrad_slabs(tokens, m);
    int st = dtype == MONARCH_F32 ? wgrad_m<float>(m, A, as, B, part, tokens, slabs, s)
                                  : wgrad_m<__nv_bfloat16>(m, A, as, B, part, tokens, slabs, s);
    if (st != MONARCH_OK) return st;
    reduce_slabs_kernel<<<(unsigned)((elems + 255) / 256), 256, 0, s>>>(part, out, elems, slabs,
                                                                       accumulate);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }
size_t esize(int dtype) { return dtype == MONARCH_F32 ? 4 : 2; }

}  // namespace

size_t staged_workspace_bytes(int op, int64_t tokens, int32_t n, int32_t m, int dtype)
{
    const size_t act = align256((size_t)tokens * n * esize(dtype));
    const size_t part = align256((size_t)wgrad_slabs(tokens, m) * m * m * m * sizeof(float));
    switch (op) {
        case MONARCH_OP_FWD:
        case MONARCH_OP_BWD_DX: return MONARCH_STATUS_BYTES + act;
        case MONARCH_OP_BWD_DW: return MONARCH_STATUS_BYTES + 2 * act + part;
        case MONARCH_OP_MLP_FWD: return MONARCH_STATUS_BYTES + 2 * act;
    }
    return 0;
}

int staged_fwd(const void *x, const void *L, const void *R, void *y, int64_t tokens, int m,
               int dtype, void *ws, cudaStream_t s)
{
    void *u = (char *)ws + MONARCH_STATUS_BYTES;   // u'[t][j*m + k] = u[t][k][j]
    MONARCH_TRY(stage(dtype, false, m, x, R, u, nullptr, 0, tokens, s));
    return stage(dtype, false, m, u, L, y, nullptr, 0, tokens, s);
}

int staged_bwd_dx(const void *dy, const void *L, const void *R, void *dx, int64_t tokens, int m,
                  int dtype, void *ws, cudaStream_t s)
{
    // du'[t][j*m + k] = sum_l L[j][l][k] dy[t][l*m + j]   (gather with P, multiply by L_j^T)
    // dx[t][k*m + i]  = sum_j R[k][j][i] du'[t][j*m + k]  (gather with P, multiply by R_k^T)
    void *du = (char *)ws + MONARCH_STATUS_BYTES;
    MONARCH_TRY(stage(dtype, true, m, dy, L, du, nullptr, 0, tokens, s));
    return stage(dtype, true, m, du, R, dx, nullptr, 0, tokens, s);
}

int staged_bwd_dw(const void *x, const void *dy, const void *L, const void *R, float *dL,
                  float *dR, int accumulate, int64_t tokens, int m, int dtype, void *ws,
                  cudaStream_t s)
{
    const size_t act = align256((size_t)tokens * m * m * esize(dtype));
    char *base = (char *)ws + MONARCH_STATUS_BYTES;
    void *u = base;                       // u'[t][j*m + k]  = u[t][k][j]
    void *du = base + act;                // du'[t][j*m + k] = du[t][k][j]
    float *part = (float *)(base + 2 * act);
    const Strides perm = {1, m};
    MONARCH_TRY(stage(dtype, false, m, x, R, u, nullptr, 0, tokens, s));
    MONARCH_TRY(stage(dtype, true, m, dy, L, du, nullptr, 0, tokens, s));
    // dL[j][l][k] = sum_t dy[t][l*m + j] u'[t][j*m + k]
    MONARCH_TRY(wgrad(dtype, m, dy, perm, u, part, dL, accumulate, tokens, s));
    // dR[k][j][i] = sum_t du'[t][j*m + k] x[t][k*m + i]
    return wgrad(dtype, m, du, perm, x, part, dR, accumulate, tokens, s);
}

int staged_mlp_fwd(const void *x, const void *L1, const void *R1, const void *b1, const void *L2,
                   const void *R2, const void *b2, void *y, int64_t tokens, int m, int dtype,
                   void *ws, cudaStream_t s)
{
    const size_t act = align256((size_t)tokens * m * m * esize(dtype));
    char *base = (char *)ws + MONARCH_STATUS_BYTES;
    void *w = base, *h = base + act;
    MONARCH_TRY(stage(dtype, false, m, x, R1, w, nullptr, 0, tokens, s));
    MONARCH_TRY(stage(dtype, false, m, w, L1, h, b1, 1, tokens, s));     // h = GELU(M1 x + b1)
    MONARCH_TRY(stage(dtype, false, m, h, R2, w, nullptr, 0, tokens, s));
    return stage(dtype, false, m, w, L2, y, b2, 0, tokens, s);           // y = M2 h + b2
}

}  // namespace monarch

// ------------------------------------------------------------------------------------------
// Forward pass for callers that cannot allocate device memory.
//
// The scratch that monarch_fwd takes from the caller's workspace (the permuted intermediate
// between the two stages) lives here in a fixed array in the library's device image, so the
// caller passes only inputs and outputs.  Every GPU that loads the library holds these
// MONARCH_NOALLOC_SCRATCH_BYTES until the process exits.
namespace monarch {
namespace {

static __device__ __align__(256) unsigned char g_noalloc_scratch[MONARCH_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void *g_noalloc_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal

// In host code `g_noalloc_scratch` is only a handle, not a device address: the address a
// kernel can use has to be asked for, once per device, while that device is current.
int noalloc_scratch_address(void **out)
{
    int dev = -1;
    MONARCH_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return MONARCH_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void *p = nullptr;
        MONARCH_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        if (!p) return MONARCH_ERR_CUDA;
        g_noalloc_ptr[dev] = p;
    }
    *out = g_noalloc_ptr[dev];
    return MONARCH_OK;
}

bool ranges_overlap(const void *a, size_t ab, const void *b, size_t bb)
{
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return ab && bb && a0 < b0 + bb && b0 < a0 + ab;
}

}  // namespace
}  // namespace monarch

extern "C" int monarch_fwd_noalloc(const void *x, const void *L, const void *R, void *y,
                                   int64_t tokens, int32_t n, int32_t m, int dtype, void *stream)
{
    using namespace monarch;
    if (tokens < 0 || n <= 0 || m <= 0 || (int64_t)m * m != (int64_t)n) return MONARCH_ERR_INVALID_ARG;
    if (dtype != MONARCH_F32 && dtype != MONARCH_BF16) return MONARCH_ERR_INVALID_ARG;
    if (m != 16 && m != 32 && m != 64 && m != 128) return MONARCH_ERR_UNSUPPORTED;
    const void *ptrs[] = {x, L, R, y};
    for (const void *p : ptrs)
        if (!p || ((uintptr_t)p & 15)) return MONARCH_ERR_INVALID_ARG;
    // the intermediate needs one element per input element; it must fit the built-in array (compared by division:
    // tokens * n * element size could wrap for absurd token counts)
    const size_t row = (size_t)n * esize(dtype);
    if ((uint64_t)tokens > (uint64_t)MONARCH_NOALLOC_SCRATCH_BYTES / row) return MONARCH_ERR_WORKSPACE;
    const size_t act = (size_t)tokens * row, wb = (size_t)n * m * esize(dtype);
    if (ranges_overlap(y, act, x, act) || ranges_overlap(y, act, L, wb) || ranges_overlap(y, act, R, wb))
        return MONARCH_ERR_INVALID_ARG;
    if (tokens == 0) return MONARCH_OK;
    void *u = nullptr;
    MONARCH_TRY(noalloc_scratch_address(&u));
    cudaStream_t s = (cudaStream_t)stream;
    // Every element of the intermediate that the second stage reads is written by the first
    // stage of this same call, so nothing left over from an earlier call is ever consumed.
    MONARCH_TRY(stage(dtype, false, m, x, R, u, nullptr, 0, tokens, s));
    return stage(dtype, false, m, u, L, y, nullptr, 0, tokens, s);
}
