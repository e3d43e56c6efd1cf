// General (rectangular) Monarch multiply y = L R x (appendix "General Monarch Matrix Parametrization", the case
// b2 = b3 = b that its block-diagonalisation theorem covers) on the CUDA cores, any sizes, both dtypes:
//   stage 1   u[t][k*b + j] = sum_i R[k][j][i]  x[t][k*b1 + i]      q blocks of b x b1, contiguous slices
//   stage 2   y[t][l*b + j] = sum_k Lp[j][l][k] u[t][k*b + j]       b blocks of r x q, slices of stride b
// Both are the same strided block product
//   out[t][blk*obs + o*oes] = sum_i W[blk][o][i] in[t][blk*ibs + i*ies],
// run by one of two kernels: a shared-memory tiled product for large blocks and, for blocks of at most 16 x 16
// (e.g. the b blocks of size 4 x 4 that stage 2 has when R has four large blocks), one thread per
// (token, block) with the block index fastest so that neighbouring threads touch neighbouring elements.
#include "common.cuh"

namespace monarch {
namespace {

struct BlockProduct {
    long long tokens;
    int nb, o, k;              // blocks, outputs and inputs per block
    int in_row, out_row;       // elements per token row
    int ibs, ies, obs, oes;    // block / element strides inside a row
    int wt;                    // 0: W[blk][o][i];  1: the block is stored transposed, W[blk][i][o] (adjoint passes)
};

constexpr int kTT = 64, kOT = 64, kKC = 16;

template <typename T>
__global__ void __launch_bounds__(256)
block_product_tiled_kernel(const T *__restrict__ in, const T *__restrict__ W, T *__restrict__ out, const BlockProduct p)
{
    __shared__ float As[kKC][kTT + 4];
    __shared__ float Bs[kKC][kOT + 4];
    const int otiles = (p.o + kOT - 1) / kOT;
    const int blk = blockIdx.y / otiles, o0 = (blockIdx.y % otiles) * kOT;
    const long long t0 = (long long)blockIdx.x * kTT;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[a][c] = 0.0f;
    const T *wb = W + (size_t)blk * p.o * p.k;
    for (int k0 = 0; k0 < p.k; k0 += kKC) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = threadIdx.x + e * 256;          // 64 rows x 16 k
            const int row = idx >> 4, kk = idx & 15;
            const long long t = t0 + row;
            float va = 0.0f, vb = 0.0f;
            if (t < p.tokens && k0 + kk < p.k)
                va = elem<T>::load(in + (size_t)t * p.in_row + (size_t)blk * p.ibs + (size_t)(k0 + kk) * p.ies);
            if (o0 + row < p.o && k0 + kk < p.k)
                vb = elem<T>::load(wb + (p.wt ? (size_t)(k0 + kk) * p.o + o0 + row : (size_t)(o0 + row) * p.k + k0 + kk));
            As[kk][row] = va;
            Bs[kk][row] = vb;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kKC; ++kk) {
            float a[4], c[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                a[e] = As[kk][ty * 4 + e];
                c[e] = Bs[kk][tx * 4 + e];
            }
#pragma unroll
            for (int e = 0; e < 4; ++e)
#pragma unroll
                for (int f = 0; f < 4; ++f) acc[e][f] = fmaf(a[e], c[f], acc[e][f]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const long long t = t0 + ty * 4 + e;
        if (t >= p.tokens) continue;
#pragma unroll
        for (int f = 0; f < 4; ++f) {
            const int o = o0 + tx * 4 + f;
            if (o < p.o) elem<T>::store(out + (size_t)t * p.out_row + (size_t)blk * p.obs + (size_t)o * p.oes, acc[e][f]);
        }
    }
}

constexpr int kSmallMax = 16;

template <typename T>
__global__ void __launch_bounds__(256)
block_product_small_kernel(const T *__restrict__ in, const T *__restrict__ W, T *__restrict__ out, const BlockProduct p)
{
    const long long total = p.tokens * p.nb;
    for (long long idx = (long long)blockIdx.x * 256 + threadIdx.x; idx < total; idx += (long long)gridDim.x * 256) {
        const long long t = idx / p.nb;
        const int blk = (int)(idx - t * p.nb);
        const T *src = in + (size_t)t * p.in_row + (size_t)blk * p.ibs;
        float v[kSmallMax];
#pragma unroll
        for (int i = 0; i < kSmallMax; ++i) v[i] = i < p.k ? elem<T>::load(src + (size_t)i * p.ies) : 0.0f;
        const T *wb = W + (size_t)blk * p.o * p.k;
        T *dst = out + (size_t)t * p.out_row + (size_t)blk * p.obs;
        for (int o = 0; o < p.o; ++o) {
            float acc = 0.0f;
#pragma unroll
            for (int i = 0; i < kSmallMax; ++i)
                if (i < p.k) acc = fmaf(elem<T>::load(wb + (p.wt ? i * p.o + o : o * p.k + i)), v[i], acc);
            elem<T>::store(dst + (size_t)o * p.oes, acc);
        }
    }
}

// Stage 2 when L's blocks are at most 4 x 4 (R has up to four large blocks): a pure streaming pass.  One thread
// owns two neighbouring columns j, keeps their two r x q blocks in registers and walks a slab of tokens; a warp
// reads and writes whole 128-byte lines (bf16) of every slice u[t][k*b + .] and y[t][l*b + .].
template <typename T> struct pair_io;
template <> struct pair_io<float> {
    static __device__ __forceinline__ float2 load(const float *p) { return *reinterpret_cast<const float2 *>(p); }
    static __device__ __forceinline__ void store(float *p, float2 v) { *reinterpret_cast<float2 *>(p) = v; }
};
template <> struct pair_io<__nv_bfloat16> {
    static __device__ __forceinline__ float2 load(const __nv_bfloat16 *p)
    {
        const uint32_t w = *reinterpret_cast<const uint32_t *>(p);
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, float2 v)
    {
        *reinterpret_cast<__nv_bfloat162 *>(p) = __floats2bfloat162_rn(v.x, v.y);
    }
};

template <typename T>
__global__ void __launch_bounds__(256)
stage2_small4_kernel(const T *__restrict__ u, const T *__restrict__ Lp, T *__restrict__ y, long long tokens, int q,
                     int b, int r, int tokens_per_slab, int wt)
{
    const int j = (blockIdx.x * 256 + threadIdx.x) * 2;
    if (j >= b) return;
    float w[2][4][4];
#pragma unroll
    for (int jj = 0; jj < 2; ++jj)
#pragma unroll
        for (int l = 0; l < 4; ++l)
#pragma unroll
            for (int k = 0; k < 4; ++k)
                w[jj][l][k] = (l < r && k < q)
                                  ? elem<T>::load(Lp + (size_t)(j + jj) * r * q + (wt ? k * r + l : l * q + k)) : 0.0f;
    const long long t0 = (long long)blockIdx.y * tokens_per_slab;
    const long long t1 = t0 + tokens_per_slab < tokens ? t0 + tokens_per_slab : tokens;
    constexpr int U = 2;                          // tokens per batch: all their loads are issued before any use
    for (long long tb = t0; tb < t1; tb += U) {
        float2 v[U][4];
#pragma unroll
        for (int tt = 0; tt < U; ++tt) {
            const T *src = u + (size_t)(tb + tt) * q * b + j;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                v[tt][k] = (k < q && tb + tt < t1) ? pair_io<T>::load(src + (size_t)k * b) : make_float2(0.0f, 0.0f);
        }
#pragma unroll
        for (int tt = 0; tt < U; ++tt) {
            if (tb + tt >= t1) break;
            T *dst = y + (size_t)(tb + tt) * r * b + j;
#pragma unroll
            for (int l = 0; l < 4; ++l) {
                if (l >= r) break;
                float2 o = make_float2(0.0f, 0.0f);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    o.x = fmaf(w[0][l][k], v[tt][k].x, o.x);
                    o.y = fmaf(w[1][l][k], v[tt][k].y, o.y);
                }
                pair_io<T>::store(dst + (size_t)l * b, o);
            }
        }
    }
}

// The same for bf16 with 16-byte accesses: a CTA owns up to 256 columns j and keeps their blocks in shared memory
// (fp32); a thread owns 8 neighbouring columns and two tokens per step, so a warp reads 512
// contiguous bytes of every slice u[t][k*b + .] and eight 16-byte loads per thread are in flight - the pass is
// bound by memory latency, not by arithmetic.
constexpr int kS2Cols = 256;

__device__ __forceinline__ float4 lds128(const float4 *p)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"((uint32_t)__cvta_generic_to_shared(p)));
    return v;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    const __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h2);
}
__device__ __forceinline__ float bf_at(const uint4 &v, int e)
{
    const uint32_t w = e < 2 ? v.x : e < 4 ? v.y : e < 6 ? v.z : v.w;
    return (e & 1) ? __uint_as_float(w & 0xFFFF0000u) : __uint_as_float(w << 16);
}

__global__ void __launch_bounds__(256, 2)
stage2_small4_bf16_kernel(const __nv_bfloat16 *__restrict__ u, const __nv_bfloat16 *__restrict__ Lp,
                          __nv_bfloat16 *__restrict__ y, long long tokens, int q, int b, int r, int tokens_per_slab, int wt)
{
    __shared__ float4 ws[4][4][2][32];            // [l][k][half][lane]: columns 8 lane + 4 half + (0..3)
    const int j0 = blockIdx.x * kS2Cols;
    for (int i = threadIdx.x; i < 16 * kS2Cols; i += 256) {
        const int jl = i >> 4, l = (i >> 2) & 3, k = i & 3;
        float v = 0.0f;
        if (j0 + jl < b && l < r && k < q) v = __bfloat162float(Lp[(size_t)(j0 + jl) * r * q + (wt ? k * r + l : l * q + k)]);
        reinterpret_cast<float *>(&ws[l][k][(jl >> 2) & 1][jl >> 3])[jl & 3] = v;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, jg = lane * 8, tr = threadIdx.x >> 5;   // 32 threads per token row, 8 rows
    if (j0 + jg >= b) return;
    const long long t0 = (long long)blockIdx.y * tokens_per_slab;
    const long long t1 = t0 + tokens_per_slab < tokens ? t0 + tokens_per_slab : tokens;
    for (long long tb = t0 + tr; tb < t1; tb += 16) {
        const bool two = tb + 8 < t1;
        uint4 v[2][4];
#pragma unroll
        for (int tt = 0; tt < 2; ++tt) {
            const __nv_bfloat16 *src = u + (size_t)(tb + tt * 8) * q * b + j0 + jg;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                v[tt][k] = (k < q && (tt == 0 || two)) ? *reinterpret_cast<const uint4 *>(src + (size_t)k * b)
                                                       : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int l = 0; l < 4; ++l) {
            if (l >= r) break;
            float acc[2][8];
#pragma unroll
            for (int tt = 0; tt < 2; ++tt)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[tt][e] = 0.0f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                // volatile: re-read per step instead of keeping all 128 weights live across the token loop
                const float4 wa = lds128(&ws[l][k][0][lane]), wb = lds128(&ws[l][k][1][lane]);
                const float wv[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
                for (int tt = 0; tt < 2; ++tt)
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[tt][e] = fmaf(wv[e], bf_at(v[tt][k], e), acc[tt][e]);
            }
#pragma unroll
            for (int tt = 0; tt < 2; ++tt) {
                if (tt == 1 && !two) break;
                const uint4 o = make_uint4(pack2(acc[tt][0], acc[tt][1]), pack2(acc[tt][2], acc[tt][3]),
                                           pack2(acc[tt][4], acc[tt][5]), pack2(acc[tt][6], acc[tt][7]));
                *reinterpret_cast<uint4 *>(y + (size_t)(tb + tt * 8) * r * b + (size_t)l * b + j0 + jg) = o;
            }
        }
    }
}

template <typename T>
int stage2_small4(const void *u, const void *Lp, void *y, long long tokens, int q, int b, int r, int wt, cudaStream_t s)
{
    const int bx = (b / 2 + 255) / 256;
    long long slabs = (148 * 8 + bx - 1) / bx;
    if (slabs > (tokens + 3) / 4) slabs = (tokens + 3) / 4;
    const int per = (int)((tokens + slabs - 1) / slabs);
    slabs = (tokens + per - 1) / per;
    if (slabs > 65535) return MONARCH_ERR_UNSUPPORTED;
    if constexpr (sizeof(T) == 2) {
        if (b % 8 == 0) {          // 16-byte accesses need rows and slices that start on 16-byte boundaries
            const int cx = (b + kS2Cols - 1) / kS2Cols;
            long long sl = (148 * 6 + cx - 1) / cx;
            if (sl > (tokens + 15) / 16) sl = (tokens + 15) / 16;
            const int pt = (int)((tokens + sl - 1) / sl);
            sl = (tokens + pt - 1) / pt;
            if (sl > 65535) return MONARCH_ERR_UNSUPPORTED;
            stage2_small4_bf16_kernel<<<dim3((unsigned)cx, (unsigned)sl), 256, 0, s>>>(
                (const __nv_bfloat16 *)u, (const __nv_bfloat16 *)Lp, (__nv_bfloat16 *)y, tokens, q, b, r, pt, wt);
            note_launch();
            MONARCH_CUDA_TRY(cudaGetLastError());
            return MONARCH_OK;
        }
    }
    {
        stage2_small4_kernel<T><<<dim3((unsigned)bx, (unsigned)slabs), 256, 0, s>>>((const T *)u, (const T *)Lp, (T *)y,
                                                                                  tokens, q, b, r, per, wt);
    }
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

// Stage 2 when L's blocks are at most 16 x 16:  y[t][l*b + j] = sum_k Lp[j][l][k] u[t][k*b + j].  A CTA owns 64
// columns j and keeps their blocks in shared memory as ws[l][k][j] (so that neighbouring threads read neighbouring
// words); a thread owns one column and walks a slab of tokens two at a time, so that every weight it reads is used
// twice.  The thread-per-(token, block) kernel above re-reads a block's q*r weights from global memory for every
// token, one 2-byte load each.
constexpr int kS2mCols = 64, kS2mLanes = 4;

template <typename T>
__global__ void __launch_bounds__(kS2mCols * kS2mLanes)
stage2_medium_kernel(const T *__restrict__ u, const T *__restrict__ Lp, T *__restrict__ y, long long tokens, int q, int b,
                     int r, int tokens_per_slab, int wt)
{
    extern __shared__ unsigned char s2m_raw[];
    T *ws = reinterpret_cast<T *>(s2m_raw);                       // [r][q][64]
    const int j0 = blockIdx.x * kS2mCols;
    for (int i = threadIdx.x; i < r * q * kS2mCols; i += kS2mCols * kS2mLanes) {
        const int jl = i / (r * q), lk = i % (r * q);               // lk = l * q + k; stored [j][l][k], or [j][k][l] if wt
        const int src = wt ? (lk % q) * r + lk / q : lk;
        ws[lk * kS2mCols + jl] = j0 + jl < b ? Lp[((size_t)(j0 + jl)) * r * q + src] : T(0.0f);
    }
    __syncthreads();
    const int jl = threadIdx.x % kS2mCols, tl = threadIdx.x / kS2mCols;
    if (j0 + jl >= b) return;
    const long long t0 = (long long)blockIdx.y * tokens_per_slab;
    const long long t1 = t0 + tokens_per_slab < tokens ? t0 + tokens_per_slab : tokens;
    for (long long ta = t0 + tl; ta < t1; ta += 2 * kS2mLanes) {
        const long long tb = ta + kS2mLanes;
        const bool two = tb < t1;
        float va[16], vb[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            va[k] = k < q ? elem<T>::load(u + (size_t)ta * q * b + (size_t)k * b + j0 + jl) : 0.0f;
            vb[k] = (k < q && two) ? elem<T>::load(u + (size_t)tb * q * b + (size_t)k * b + j0 + jl) : 0.0f;
        }
        for (int l = 0; l < r; ++l) {
            float xa = 0.0f, xb = 0.0f;
#pragma unroll
            for (int k = 0; k < 16; ++k)
                if (k < q) {
                    const float w = elem<T>::load(ws + (l * q + k) * kS2mCols + jl);
                    xa = fmaf(w, va[k], xa);
                    xb = fmaf(w, vb[k], xb);
                }
            elem<T>::store(y + (size_t)ta * r * b + (size_t)l * b + j0 + jl, xa);
            if (two) elem<T>::store(y + (size_t)tb * r * b + (size_t)l * b + j0 + jl, xb);
        }
    }
}

template <typename T>
int stage2_medium(const void *u, const void *Lp, void *y, long long tokens, int q, int b, int r, int wt, cudaStream_t s)
{
    const int cx = (b + kS2mCols - 1) / kS2mCols;
    long long slabs = (148 * 8 + cx - 1) / cx;
    if (slabs > (tokens + 7) / 8) slabs = (tokens + 7) / 8;
    const int per = (int)((tokens + slabs - 1) / slabs);
    slabs = (tokens + per - 1) / per;
    if (slabs > 65535) return MONARCH_ERR_UNSUPPORTED;
    const int smem = r * q * kS2mCols * (int)sizeof(T);           // at most 64 KB (fp32, 16 x 16)
    static bool attr = false;
    if (!attr) {
        MONARCH_CUDA_TRY(cudaFuncSetAttribute(stage2_medium_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              16 * 16 * kS2mCols * (int)sizeof(T)));
        attr = true;
    }
    stage2_medium_kernel<T><<<dim3((unsigned)cx, (unsigned)slabs), kS2mCols * kS2mLanes, smem, s>>>(
        (const T *)u, (const T *)Lp, (T *)y, tokens, q, b, r, per, wt);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

template <typename T>
int block_product(const void *in, const void *W, void *out, const BlockProduct &p, cudaStream_t s)
{
    if (p.tokens == 0 || p.nb == 0 || p.o == 0) return MONARCH_OK;
    if (p.o <= kSmallMax && p.k <= kSmallMax) {
        long long blocks = (p.tokens * p.nb + 255) / 256;
        if (blocks > 148 * 32) blocks = 148 * 32;
        block_product_small_kernel<T><<<(unsigned)blocks, 256, 0, s>>>((const T *)in, (const T *)W, (T *)out, p);
    } else {
        const long long gx = (p.tokens + kTT - 1) / kTT;
        const long long gy = (long long)p.nb * ((p.o + kOT - 1) / kOT);
        if (gx > 0x7fffffffLL || gy > 65535) return MONARCH_ERR_UNSUPPORTED;
        block_product_tiled_kernel<T><<<dim3((unsigned)gx, (unsigned)gy), 256, 0, s>>>((const T *)in, (const T *)W,
                                                                                     (T *)out, p);
    }
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

}  // namespace

size_t rect_workspace_bytes(int64_t tokens, int q, int b, int dtype)
{
    const size_t es = dtype == MONARCH_F32 ? 4 : 2;
    return MONARCH_STATUS_BYTES + (((size_t)tokens * q * b * es + 255) & ~(size_t)255);
}

// wt = 0: u = blockdiag(R) x.  wt = 1: the adjoint, dx = blockdiag(R)^T du (pass du as x; b1 and b swap roles).
int rect_stage1_simt(const void *x, const void *R, void *u, int64_t tokens, int q, int b1, int b, int dtype, int wt,
                     cudaStream_t s)
{
    const BlockProduct s1 = {tokens, q, b, b1, q * b1, q * b, b1, 1, b, 1, wt};
    return dtype == MONARCH_F32 ? block_product<float>(x, R, u, s1, s) : block_product<__nv_bfloat16>(x, R, u, s1, s);
}

// wt = 0: y[t][l*b + j] = sum_k Lp[j][l][k] u[t][k*b + j] (q slices in, r out).  wt = 1: the adjoint,
// du[t][k*b + j] = sum_l Lp[j][l][k] dy[t][l*b + j]: call with q = r of the forward, r = q of the forward.
int rect_stage2_simt(const void *u, const void *Lp, void *y, int64_t tokens, int q, int b, int r, int dtype, int wt,
                     cudaStream_t s)
{
    const BlockProduct s2 = {tokens, b, r, q, q * b, r * b, 1, b, 1, b, wt};
    const bool small4 = q <= 4 && r <= 4 && b % 2 == 0 && tokens > 0;
    const bool medium = !small4 && q <= 16 && r <= 16 && b >= 32 && tokens > 0;
    if (dtype == MONARCH_F32)
        return small4   ? stage2_small4<float>(u, Lp, y, tokens, q, b, r, wt, s)
               : medium ? stage2_medium<float>(u, Lp, y, tokens, q, b, r, wt, s)
                        : block_product<float>(u, Lp, y, s2, s);
    return small4   ? stage2_small4<__nv_bfloat16>(u, Lp, y, tokens, q, b, r, wt, s)
           : medium ? stage2_medium<__nv_bfloat16>(u, Lp, y, tokens, q, b, r, wt, s)
                    : block_product<__nv_bfloat16>(u, Lp, y, s2, s);
}

// ---------------------------------------------------------------------------------------------------------
// Token reductions of the backward pass:  out[blk][o][i] (+)= sum_t A[t][blk*abs + o*aes] * B[t][blk*bbs + i*bes]
//   dL[j][l][k] = sum_t dy[t][l*b + j] u[t][k*b + j]      (blk = j: strides 1 / b)
//   dR[k][j][i] = sum_t du[t][k*b + j] x[t][k*b1 + i]     (blk = k: strides b / 1 and b1 / 1)
// fp32 partial sums per token slab, added to the fp32 output with atomics (summation order may vary run to run).
namespace {

struct TokenReduce {
    long long tokens;
    int nb, o, k;
    int a_row, b_row;
    int abs_, aes, bbs, bes;
    int tokens_per_slab;
};

// large blocks: a CTA owns a 64 x 64 tile of one block's gradient and a slab of tokens (tokens are the GEMM's K)
template <typename T>
__global__ void __launch_bounds__(256)
token_reduce_tiled_kernel(const T *__restrict__ A, const T *__restrict__ B, float *__restrict__ out, const TokenReduce p)
{
    __shared__ float As[kKC][kTT + 4];
    __shared__ float Bs[kKC][kOT + 4];
    const int otiles = (p.o + 63) / 64, ktiles = (p.k + 63) / 64;
    const int blk = blockIdx.x / (otiles * ktiles), rem = blockIdx.x % (otiles * ktiles);
    const int o0 = (rem / ktiles) * 64, k0 = (rem % ktiles) * 64;
    const long long t0 = (long long)blockIdx.y * p.tokens_per_slab;
    const long long t1 = t0 + p.tokens_per_slab < p.tokens ? t0 + p.tokens_per_slab : p.tokens;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[a][c] = 0.0f;
    for (long long tb = t0; tb < t1; tb += kKC) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = threadIdx.x + e * 256;           // 16 tokens x 64 columns
            const int tt = idx >> 6, c = idx & 63;
            const long long t = tb + tt;
            float va = 0.0f, vb = 0.0f;
            if (t < t1 && o0 + c < p.o)
                va = elem<T>::load(A + (size_t)t * p.a_row + (size_t)blk * p.abs_ + (size_t)(o0 + c) * p.aes);
            if (t < t1 && k0 + c < p.k)
                vb = elem<T>::load(B + (size_t)t * p.b_row + (size_t)blk * p.bbs + (size_t)(k0 + c) * p.bes);
            As[tt][c] = va;
            Bs[tt][c] = vb;
        }
        __syncthreads();
#pragma unroll
        for (int tt = 0; tt < kKC; ++tt) {
            float a[4], c[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                a[e] = As[tt][ty * 4 + e];
                c[e] = Bs[tt][tx * 4 + e];
            }
#pragma unroll
            for (int e = 0; e < 4; ++e)
#pragma unroll
                for (int f = 0; f < 4; ++f) acc[e][f] = fmaf(a[e], c[f], acc[e][f]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int f = 0; f < 4; ++f) {
            const int o = o0 + ty * 4 + e, k = k0 + tx * 4 + f;
            if (o < p.o && k < p.k) atomicAdd(out + ((size_t)blk * p.o + o) * p.k + k, acc[e][f]);
        }
}

// blocks of at most 16 x 16: one thread per (block, output row), block index fastest
template <typename T>
__global__ void __launch_bounds__(256)
token_reduce_small_kernel(const T *__restrict__ A, const T *__restrict__ B, float *__restrict__ out, const TokenReduce p)
{
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    if (idx >= (long long)p.nb * p.o) return;
    const int o = (int)(idx / p.nb), blk = (int)(idx % p.nb);
    const long long t0 = (long long)blockIdx.y * p.tokens_per_slab;
    const long long t1 = t0 + p.tokens_per_slab < p.tokens ? t0 + p.tokens_per_slab : p.tokens;
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.0f;
    for (long long t = t0; t < t1; ++t) {
        const float a = elem<T>::load(A + (size_t)t * p.a_row + (size_t)blk * p.abs_ + (size_t)o * p.aes);
        const T *brow = B + (size_t)t * p.b_row + (size_t)blk * p.bbs;
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (i < p.k) acc[i] = fmaf(a, elem<T>::load(brow + (size_t)i * p.bes), acc[i]);
    }
    if (t1 > t0) {
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (i < p.k) atomicAdd(out + ((size_t)blk * p.o + o) * p.k + i, acc[i]);
    }
}

// dL[j][l][k] += sum_t dy[t][l*b + j] u[t][k*b + j] for blocks of at most 4 x 4: one thread owns two neighbouring
// columns j and their 2 x 16 partial sums, walks a slab of tokens with 4-byte loads (a warp reads whole 128-byte
// lines of every slice), and adds its sums to the output once.
template <typename T>
__global__ void __launch_bounds__(256)
dl_small4_kernel(const T *__restrict__ dy, const T *__restrict__ u, float *__restrict__ dL, long long tokens, int q, int b,
                 int r, int tokens_per_slab)
{
    const int j = (blockIdx.x * 256 + threadIdx.x) * 2;
    if (j >= b) return;
    float acc[2][4][4];
#pragma unroll
    for (int jj = 0; jj < 2; ++jj)
#pragma unroll
        for (int l = 0; l < 4; ++l)
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[jj][l][k] = 0.0f;
    const long long t0 = (long long)blockIdx.y * tokens_per_slab;
    const long long t1 = t0 + tokens_per_slab < tokens ? t0 + tokens_per_slab : tokens;
#pragma unroll 2
    for (long long t = t0; t < t1; ++t) {
        float2 g[4], v[4];
#pragma unroll
        for (int l = 0; l < 4; ++l)
            g[l] = l < r ? pair_io<T>::load(dy + (size_t)t * r * b + (size_t)l * b + j) : make_float2(0.0f, 0.0f);
#pragma unroll
        for (int k = 0; k < 4; ++k)
            v[k] = k < q ? pair_io<T>::load(u + (size_t)t * q * b + (size_t)k * b + j) : make_float2(0.0f, 0.0f);
#pragma unroll
        for (int l = 0; l < 4; ++l)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[0][l][k] = fmaf(g[l].x, v[k].x, acc[0][l][k]);
                acc[1][l][k] = fmaf(g[l].y, v[k].y, acc[1][l][k]);
            }
    }
    if (t1 > t0) {
#pragma unroll
        for (int jj = 0; jj < 2; ++jj)
#pragma unroll
            for (int l = 0; l < 4; ++l)
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (l < r && k < q) atomicAdd(dL + ((size_t)(j + jj) * r + l) * q + k, acc[jj][l][k]);
    }
}

template <typename T>
int dl_small4(const void *dy, const void *u, float *dL, long long tokens, int q, int b, int r, cudaStream_t s)
{
    const int bx = (b / 2 + 255) / 256;
    long long slabs = (148 * 4 + bx - 1) / bx;
    if (slabs > (tokens + 31) / 32) slabs = (tokens + 31) / 32;
    const int per = (int)((tokens + slabs - 1) / slabs);
    slabs = (tokens + per - 1) / per;
    if (slabs > 65535) return MONARCH_ERR_UNSUPPORTED;
    dl_small4_kernel<T><<<dim3((unsigned)bx, (unsigned)slabs), 256, 0, s>>>((const T *)dy, (const T *)u, dL, tokens, q, b, r, per);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

template <typename T>
int token_reduce(const void *A, const void *B, float *out, TokenReduce p, cudaStream_t s)
{
    if (p.tokens == 0 || p.nb == 0) return MONARCH_OK;
    if (p.o <= 16 && p.k <= 16) {
        const long long bx = ((long long)p.nb * p.o + 255) / 256;
        long long slabs = (148 * 8 + bx - 1) / bx;
        if (slabs > (p.tokens + 31) / 32) slabs = (p.tokens + 31) / 32;
        p.tokens_per_slab = (int)((p.tokens + slabs - 1) / slabs);
        slabs = (p.tokens + p.tokens_per_slab - 1) / p.tokens_per_slab;
        if (bx > 0x7fffffffLL || slabs > 65535) return MONARCH_ERR_UNSUPPORTED;
        token_reduce_small_kernel<T><<<dim3((unsigned)bx, (unsigned)slabs), 256, 0, s>>>((const T *)A, (const T *)B, out, p);
    } else {
        const long long bx = (long long)p.nb * ((p.o + 63) / 64) * ((p.k + 63) / 64);
        long long slabs = (148 * 4 + bx - 1) / bx;
        if (slabs > (p.tokens + 255) / 256) slabs = (p.tokens + 255) / 256;
        if (slabs < 1) slabs = 1;
        p.tokens_per_slab = (int)((p.tokens + slabs - 1) / slabs);
        p.tokens_per_slab = (p.tokens_per_slab + kKC - 1) / kKC * kKC;
        slabs = (p.tokens + p.tokens_per_slab - 1) / p.tokens_per_slab;
        if (bx > 0x7fffffffLL || slabs > 65535) return MONARCH_ERR_UNSUPPORTED;
        token_reduce_tiled_kernel<T><<<dim3((unsigned)bx, (unsigned)slabs), 256, 0, s>>>((const T *)A, (const T *)B, out, p);
    }
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

}  // namespace

// dL += sum_t dy (x) u  and  dR += sum_t du (x) x  (the caller zeroes them first when not accumulating)
int rect_wgrad_simt(const void *x, const void *dy, const void *u, const void *du, float *dL, float *dR, int64_t tokens,
                    int q, int b1, int b, int r, int dtype, int want_dL, int want_dR, cudaStream_t s)
{
    const TokenReduce gl = {tokens, b, r, q, r * b, q * b, 1, b, 1, b, 0};
    const TokenReduce gr = {tokens, q, b, b1, q * b, q * b1, b, 1, b1, 1, 0};
    const bool small4 = q <= 4 && r <= 4 && b % 2 == 0 && tokens > 0;
    if (dtype == MONARCH_F32) {
        if (want_dL)
            MONARCH_TRY(small4 ? dl_small4<float>(dy, u, dL, tokens, q, b, r, s) : token_reduce<float>(dy, u, dL, gl, s));
        return want_dR ? token_reduce<float>(du, x, dR, gr, s) : MONARCH_OK;
    }
    if (want_dL)
        MONARCH_TRY(small4 ? dl_small4<__nv_bfloat16>(dy, u, dL, tokens, q, b, r, s)
                           : token_reduce<__nv_bfloat16>(dy, u, dL, gl, s));
    return want_dR ? token_reduce<__nv_bfloat16>(du, x, dR, gr, s) : MONARCH_OK;
}

}  // namespace monarch
