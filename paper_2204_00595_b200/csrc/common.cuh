// Shared host/device helpers of libmonarch (internal; not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "monarch.h"

namespace monarch {

// Launch counter behind monarch_launch_count().
void note_launch(int n = 1);

// SM count of the current device (cached per device ordinal, safe against concurrent first calls).
int current_device_sms(int *sms);

// A value cached per device ordinal (an occupancy figure): get() returns -1 until set() has stored one for the current
// device.  Two threads racing on a first call both compute and store the same value.
struct PerDeviceCache {
    std::atomic<int> v[64];                  // value + 1; zero-initialised as a static
    int get() const
    {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
        return v[dev].load(std::memory_order_relaxed) - 1;
    }
    void set(int value)
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) v[dev].store(value + 1, std::memory_order_relaxed);
    }
};

#define MONARCH_CUDA_TRY(expr)                                   \
    do {                                                         \
        cudaError_t err_ = (expr);                               \
        if (err_ != cudaSuccess) return MONARCH_ERR_CUDA;        \
    } while (0)

#define MONARCH_TRY(expr)                                        \
    do {                                                         \
        int st_ = (expr);                                        \
        if (st_ != MONARCH_OK) return st_;                       \
    } while (0)

template <typename T> struct elem;
template <> struct elem<float> {
    static __device__ __forceinline__ float load(const float *p) { return *p; }
    static __device__ __forceinline__ void store(float *p, float v) { *p = v; }
};
template <> struct elem<__nv_bfloat16> {
    static __device__ __forceinline__ float load(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }
};

// erf form of GELU, evaluated in fp32.
static __device__ __forceinline__ float gelu_erf(float a)
{
    return 0.5f * a * (1.0f + erff(a * 0.70710678118654752440f));
}

// GELU(a) = a/2 (1 + erf(a / sqrt 2)) evaluated as a * sigmoid(2 a (c0 + c1 a^2 + c2 a^4)): the logistic form
// of the usual tanh approximation with one more polynomial term, coefficients fitted (minimax over [-8, 8]) to
// the erf definition: |error| <= 2.6e-5 everywhere (a^2 is clamped at 64, beyond which the sigmoid has
// saturated) - well below one bf16 ulp of the result.  Nine instructions, two of them MUFU; the libm-grade erf
// costs twice that.  Used where the result is rounded to bf16 anyway; fp32 paths use gelu_erf.
static __device__ __forceinline__ float gelu_fast_exp(float a)               // exp(-2 a poly(a^2))
{
    const float a2 = fminf(a * a, 64.0f);
    float t = fmaf(a2, 0.0010142630198970437f, -0.10677572339773178f);     // -2 log2(e) * (c2 a^2 + c1)
    t = fmaf(a2, t, -2.301121234893799f);
    // flush-to-zero forms: no range fix-up code around the two MUFU operations (the exponent is at most 40 for
    // |a| <= 8; beyond that 2^x overflows to inf or flushes to 0 and the sigmoid saturates to 0 or 1, as it should)
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(a * t));
    return e;
}
static __device__ __forceinline__ float gelu_fast(float a)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + gelu_fast_exp(a)));
    return a * r;
}

// d/da GELU(a) = Phi(a) + a phi(a) with Phi from the same sigmoid (|Phi error| <= 5.1e-5) and the normal
// density phi evaluated directly: |error| <= 5.1e-5, for results that are rounded to bf16.
static __device__ __forceinline__ float gelu_fast_grad(float a)
{
    const float pdf = 0.39894228040143267794f * exp2f(-0.72134752044448170368f * a * a);
    return fmaf(a, pdf, __fdividef(1.0f, 1.0f + gelu_fast_exp(a)));
}

// ---- staged (one block-diagonal stage per launch) kernels, staged_simt.cu ----
// Workspace layout helpers and launchers; every launcher returns a monarch_status_t.
size_t staged_workspace_bytes(int op, int64_t tokens, int32_t n, int32_t m, int dtype);
int staged_fwd(const void *x, const void *L, const void *R, void *y, int64_t tokens, int m,
               int dtype, void *ws, cudaStream_t s);
int staged_bwd_dx(const void *dy, const void *L, const void *R, void *dx, int64_t tokens, int m,
                  int dtype, void *ws, cudaStream_t s);
int staged_bwd_dw(const void *x, const void *dy, const void *L, const void *R, float *dL,
                  float *dR, int accumulate, int64_t tokens, int m, int dtype, void *ws,
                  cudaStream_t s);
int staged_mlp_fwd(const void *x, const void *L1, const void *R1, const void *b1, const void *L2,
                   const void *R2, const void *b2, void *y, int64_t tokens, int m, int dtype,
                   void *ws, cudaStream_t s);


// ---- tensor-core stage chains through the workspace (bf16, m >= 32), tc_stage.cu ----
int tc_staged_fwd(const void *x, const void *L, const void *R, void *y, int64_t tokens, int m,
                  void *ws, cudaStream_t s);
int tc_staged_mlp_fwd(const void *x, const void *L1, const void *R1, const void *b1, const void *L2,
                      const void *R2, const void *b2, void *y, int64_t tokens, int m, void *ws,
                      cudaStream_t s);


// m = 128 as chains of block GEMMs on token-innermost planes (chain_m128.cu)
size_t chain_fwd_m128_workspace_bytes(int64_t tokens);
size_t chain_bwd_m128_workspace_bytes(int64_t tokens);
int chain_fwd_m128(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws, cudaStream_t s);
// saved_up: the u' the forward call left in its workspace (chain_fwd_m128_saved_u), or null
int chain_bwd_m128(const void *x, const void *dy, const void *L, const void *R, const void *saved_up, void *dx, float *dL,
                   float *dR, int accumulate, int want_dx, int want_dw, int64_t tokens, void *ws, cudaStream_t s);
const void *chain_fwd_m128_saved_u(const void *fwd_ws, int64_t tokens);
// test aid: the next plane-transpose launch (last step of the m = 128 forward) leaves out the load of this item
void debug_skip_next_plane_load(long long item);

// ---- backward as a chain of tensor-core launches (bf16; dx for m >= 32, dL/dR for m = 128), tc_bwd.cu ----
// fixed_order (m = 32, 64): kTcPartialBytes more; the token slices of the weight-gradient launches store their sums there and a
// small launch adds them in slice order (same bits on every run) instead of reductions in L2
constexpr size_t kTcPartialBytes = (size_t)32 << 20;
size_t tc_staged_bwd_workspace_bytes(int64_t tokens, int m, bool fixed_order = false);
// saved_up: for m = 128, the u' planes left by the forward call (chain_fwd_m128_saved_u), or null
int tc_staged_bwd(const void *x, const void *dy, const void *L, const void *R, void *dx, float *dL, float *dR,
                  int accumulate, int want_dx, int want_dw, int64_t tokens, int m, void *ws, cudaStream_t s,
                  const void *saved_up = nullptr, bool fixed_order = false);

// ---- forward for m = 16 in one launch on the CUDA cores, both dtypes (fused_m16.cu); no workspace use ----
int fused_fwd_m16(const void *x, const void *L, const void *R, void *y, int64_t tokens, int dtype, cudaStream_t s);

// ---- fused forward for m = 32, bf16: both stages inside one CTA (fused_m32.cu); workspace = status word only ----
int fused_fwd_m32(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws, cudaStream_t s);

// ---- fused single-pass forward for m = 64, bf16 (fused_m64.cu) ----
size_t fused_fwd_m64_workspace_bytes(int64_t tokens);
int fused_fwd_m64(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws,
                  cudaStream_t s);
// the same on clusters of four CTAs with the intermediate in distributed shared memory (fused_m64_cluster.cu);
// MONARCH_ERR_UNSUPPORTED when the device cannot host such a cluster
int fused_fwd_m64_cluster(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws, cudaStream_t s);
bool fused_fwd_m64_on_clusters();
// the same with every CTA doing both stages (fused_m64_team.cu); same workspace layout
int fused_fwd_m64_team(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws,
                       cudaStream_t s);
// feed-forward block as two passes of the team kernel with bias (+ GELU) in the stage-2 epilogue
size_t fused_mlp_fwd_m64_workspace_bytes(int64_t tokens);
int fused_mlp_fwd_m64(const void *x, const void *L1, const void *R1, const void *b1, const void *L2,
                      const void *R2, const void *b2, void *y, int64_t tokens, void *ws, cudaStream_t s);
// one pass y = act(M x + bias), act = GELU or identity; workspace layout of fused_fwd_m64 (u stays behind)
int fused_fwd_bias_m64(const void *x, const void *L, const void *R, const void *bias, int gelu, void *y,
                       int64_t tokens, void *ws, cudaStream_t s);
// first stage only: u = P R x in the exchange layout [tile][j][k/8][t%64][k%8] (tokens rounded up to 64)
int fused_fwd_m64_stage1(const void *x, const void *R, void *u, int64_t tokens, unsigned *status,
                         cudaStream_t s);

// ---- fused single-pass dx = M^T dy for m = 64, bf16 (fused_m64_bwd.cu) ----
size_t fused_bwd_dx_m64_workspace_bytes(int64_t tokens);
int fused_bwd_dx_m64(const void *dy, const void *L, const void *R, void *dx, int64_t tokens, void *ws,
                     cudaStream_t s);
// first stage only: du as [tile][k][j/8][t%64][j%8] and P dy as [tile][j][l/8][t%64][l%8]
int fused_bwd_m64_stage1(const void *dy, const void *L, void *du, void *dyp, int64_t tokens,
                         unsigned *status, cudaStream_t s);

// both stages, also leaving du (and P dy if dyp != null) behind for the weight gradients
int fused_bwd_dx_m64_keep(const void *dy, const void *L, const void *R, void *dx, void *du, void *dyp,
                          unsigned *counters, unsigned *status, int64_t tokens, cudaStream_t s);

// dx, dL +=, dR += in one launch; u = P R x in the forward exchange layout, du / dyp = scratch exchange buffers
// partials (optional, kBwdPartialBytes): per-CTA partial sums + a fixed-order reduction instead of atomic adds; dL, dR
// are then overwritten (accumulate = 0) or added to (1) by that reduction
constexpr int kBwdMaxPartials = 16;                                  // CTAs per group of a weight-gradient kind, at most
constexpr size_t kBwdPartialBytes = (size_t)2 * kBwdMaxPartials * 64 * 64 * 64 * sizeof(float);
int fused_bwd_all_m64(const void *x, const void *dy, const void *L, const void *R, const void *u, void *dx,
                      void *du, void *dyp, float *dL, float *dR, unsigned *counters, unsigned *status,
                      int64_t tokens, cudaStream_t s, float *partials = nullptr, int accumulate = 1);

// ---- weight gradients for m = 64, bf16 (fused_m64_bwd_dw.cu) ----
// fixed_order: the weight gradients are summed in a fixed order (partial sums in the workspace, which is then
// kBwdPartialBytes larger); refused (MONARCH_ERR_UNSUPPORTED) where the one-launch backward cannot run
size_t fused_bwd_dw_m64_workspace_bytes(int64_t tokens, bool fixed_order = false);
int fused_bwd_dw_m64(const void *x, const void *dy, const void *L, const void *R, float *dL, float *dR,
                     int accumulate, int64_t tokens, void *ws, cudaStream_t s, bool fixed_order = false);
// dx, dL, dR in one pass; u_saved (optional) = the exchange buffer a fused forward call left behind
size_t fused_bwd_m64_workspace_bytes(int64_t tokens, bool fixed_order = false);
int fused_bwd_m64(const void *x, const void *dy, const void *L, const void *R, const void *u_saved,
                  void *dx, float *dL, float *dR, int accumulate, int64_t tokens, void *ws,
                  cudaStream_t s, bool fixed_order = false);
// where the fused forward keeps u inside its workspace
const void *fused_fwd_m64_saved_u(const void *fwd_ws);

// ---- general (rectangular) Monarch multiply on the CUDA cores (rect_simt.cu); workspace = [status][u] ----
size_t rect_workspace_bytes(int64_t tokens, int q, int b, int dtype);
// wt = 1 reads the blocks transposed (the adjoint passes of the backward call)
int rect_stage1_simt(const void *x, const void *R, void *u, int64_t tokens, int q, int b1, int b, int dtype, int wt,
                     cudaStream_t s);
int rect_stage2_simt(const void *u, const void *Lp, void *y, int64_t tokens, int q, int b, int r, int dtype, int wt,
                     cudaStream_t s);
// want_dL / want_dR = 0: that gradient comes from the streaming pass / the tensor-core kernel
int rect_wgrad_simt(const void *x, const void *dy, const void *u, const void *du, float *dL, float *dR, int64_t tokens,
                    int q, int b1, int b, int r, int dtype, int want_dL, int want_dR, cudaStream_t s);
// stage 1 on the tensor cores (rect_tc.cu): bf16, b1 and b multiples of 64
bool rect_stage1_tc_available(int q, int b1, int b, int dtype);
int rect_stage1_tc(const void *x, const void *R, void *u, int64_t tokens, int q, int b1, int b, unsigned *status,
                   cudaStream_t s);
int rect_stage1_adjoint_tc(const void *du, const void *R, void *dx, int64_t tokens, int q, int b1, int b,
                           unsigned *status, cudaStream_t s);
// dL for blocks up to 4 x 4 as a TMA-fed streaming pass (rect_tc.cu): sizes as rect_stage2_stream_available
int rect_dl_stream(const void *dy, const void *u, float *dL, int64_t tokens, int q, int b, int r, unsigned *status,
                   cudaStream_t s);
bool rect_wgrad_R_tc_available(int q, int b1, int b, int dtype);
int rect_wgrad_R_tc(const void *du, const void *x, float *dR, int64_t tokens, int q, int b1, int b, unsigned *status,
                    cudaStream_t s);
// stage 2 as a TMA-fed streaming pass (rect_tc.cu): bf16, q and r at most 4, b a multiple of 8 and at least 256
bool rect_stage2_stream_available(int q, int b, int r, int dtype);
int rect_stage2_stream(const void *u, const void *Lp, void *y, int64_t tokens, int q, int b, int r, int wt,
                       unsigned *status, cudaStream_t s);

// ---- rectangular class with wrapped-diagonal blocks, b2 != b3 (rect_wrapped.cu) ----
size_t rectw_workspace_bytes(int64_t tokens, int q, int b2, int b3, int r, int dtype);
size_t rectw_bwd_workspace_bytes(int64_t tokens, int q, int b2, int b3, int r, int dtype);
int rectw_fwd(const void *x, const void *Lw, const void *R, void *y, int64_t tokens, int q, int b1, int b2, int b3, int r,
              int dtype, bool fast, void *ws, cudaStream_t s);
int rectw_bwd(const void *x, const void *dy, const void *Lw, const void *R, void *dx, float *dLw, float *dR, int accumulate,
              int64_t tokens, int q, int b1, int b2, int b3, int r, int dtype, bool fast, void *ws, cudaStream_t s);

// ---- dense <-> Monarch factors (project.cu): Eq. (2) and Algorithm 1 ----
int dense_from_factors(const void *L, const void *R, void *M, int m, int dtype, cudaStream_t s);
int project_to_factors(const void *A, void *L, void *R, int m, int dtype, unsigned long long *rotations, cudaStream_t s);

// ---- elementwise steps of the feed-forward block's backward pass (mlp_bwd.cu) ----
// h = GELU(a (+ b1)); b1 may be null when a already holds the bias
int mlp_act(const void *a, const void *b1, void *h, int64_t tokens, int n, int dtype, cudaStream_t s);
// dh <- dh * GELU'(a (+ b1)) in place, db1 += column sums of the result, db2 += column sums of dy
int mlp_dact(void *dh, const void *a, const void *b1, const void *dy, float *db1, float *db2, int64_t tokens, int n,
             int dtype, cudaStream_t s);
// combination step of the complex multiply (planar tensors, plane_elems = tokens * n)
int cplx_combine(const void *A, const void *B, const void *C, const void *D, void *y, int64_t plane_elems, int adjoint,
                 int dtype, cudaStream_t s);
// fold the status word of an inner workspace into the outer one and clear it
int merge_status(unsigned *outer, unsigned *inner, cudaStream_t s);

}  // namespace monarch
