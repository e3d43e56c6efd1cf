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
            if (o0 + row < p.o && k0 + kk < p.k) vb = elem<T>::load(wb + (size_t)(o0 + row) * p.k + k0 + kk);
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
                if (i < p.k) acc = fmaf(elem<T>::load(wb + o * p.k + i), v[i], acc);
            elem<T>::store(dst + (size_t)o * p.oes, acc);
        }
    }
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

int rect_fwd_simt(const void *x, const void *Lp, const void *R, void *y, int64_t tokens, int q, int b1, int b, int r,
                  int dtype, void *ws, int stage1_done, cudaStream_t s)
{
    void *u = (char *)ws + MONARCH_STATUS_BYTES;
    const BlockProduct s1 = {tokens, q, b, b1, q * b1, q * b, b1, 1, b, 1};
    const BlockProduct s2 = {tokens, b, r, q, q * b, r * b, 1, b, 1, b};
    if (dtype == MONARCH_F32) {
        if (!stage1_done) MONARCH_TRY(block_product<float>(x, R, u, s1, s));
        return block_product<float>(u, Lp, y, s2, s);
    }
    if (!stage1_done) MONARCH_TRY(block_product<__nv_bfloat16>(x, R, u, s1, s));
    return block_product<__nv_bfloat16>(u, Lp, y, s2, s);
}

}  // namespace monarch
