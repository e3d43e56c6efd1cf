// Forward y = P L P^T R x for m = 16 (n = 256) in one launch on the CUDA cores, fp32 or bf16 storage with fp32
// arithmetic.  A token vector is 256 elements, so a CTA keeps a few tokens and their intermediate u' in shared
// memory and runs both stages of Section 3.3 (steps 1-3) back to back: thread e = j*16 + k forms
// u'[t][j][k] = sum_i R[k][j][i] x[t][k*16+i] with its row of R in registers, then thread e = l*16 + j forms
// y[t][l*16+j] = sum_k L[j][l][k] u'[t][j][k].  At this size the two-launch chain is bound by launch latency;
// one launch halves it.  (Blocks of 16 x 16 are below the tensor-core tile: fp32 FMA is the right unit, and in
// fp32 mode the only one that meets the 1e-5 tolerance.)
#include "common.cuh"

namespace monarch {
namespace {

constexpr int kM16 = 16, kN16 = 256;

template <typename T, int TOK>
__global__ void __launch_bounds__(kN16) fused_fwd_m16_kernel(const T *__restrict__ x, const T *__restrict__ L,
                                                             const T *__restrict__ R, T *__restrict__ y,
                                                             long long tokens)
{
    __shared__ float xs[TOK][kN16];
    __shared__ float us[TOK][kN16 + 1];
    const int e = threadIdx.x;
    const long long t0 = (long long)blockIdx.x * TOK;
    const int nt = tokens - t0 < TOK ? (int)(tokens - t0) : TOK;

    for (int t = 0; t < nt; ++t) xs[t][e] = elem<T>::load(x + (t0 + t) * kN16 + e);

    // both rows of weights are requested before the first barrier: one trip to memory instead of two in a row
    float wl[kM16];
    {
        const int l = e >> 4, j = e & 15;
#pragma unroll
        for (int k = 0; k < kM16; ++k) wl[k] = elem<T>::load(L + (j * kM16 + l) * kM16 + k);
    }
    // stage 1: e = j*16 + k
    {
        const int j = e >> 4, k = e & 15;
        float w[kM16];
#pragma unroll
        for (int i = 0; i < kM16; ++i) w[i] = elem<T>::load(R + (k * kM16 + j) * kM16 + i);
        __syncthreads();
        for (int t = 0; t < nt; ++t) {
            float acc = 0.f;
#pragma unroll
            for (int i = 0; i < kM16; ++i) acc = fmaf(w[i], xs[t][k * kM16 + i], acc);
            us[t][e] = acc;
        }
    }
    // stage 2: e = l*16 + j
    {
        const int j = e & 15;
        __syncthreads();
        for (int t = 0; t < nt; ++t) {
            float acc = 0.f;
#pragma unroll
            for (int k = 0; k < kM16; ++k) acc = fmaf(wl[k], us[t][j * kM16 + k], acc);
            elem<T>::store(y + (t0 + t) * kN16 + e, acc);
        }
    }
}

template <typename T>
int launch_m16(const void *x, const void *L, const void *R, void *y, int64_t tokens, cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    // few tokens: small tiles so that many SMs share the latency; many tokens: amortise the weight reads
    if (tokens <= 4096) {
        fused_fwd_m16_kernel<T, 4><<<(unsigned)((tokens + 3) / 4), kN16, 0, s>>>((const T *)x, (const T *)L, (const T *)R,
                                                                               (T *)y, tokens);
    } else {
        fused_fwd_m16_kernel<T, 16><<<(unsigned)((tokens + 15) / 16), kN16, 0, s>>>((const T *)x, (const T *)L,
                                                                                 (const T *)R, (T *)y, tokens);
    }
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

}  // namespace

int fused_fwd_m16(const void *x, const void *L, const void *R, void *y, int64_t tokens, int dtype, cudaStream_t s)
{
    return dtype == MONARCH_F32 ? launch_m16<float>(x, L, R, y, tokens, s)
                                : launch_m16<__nv_bfloat16>(x, L, R, y, tokens, s);
}

}  // namespace monarch
