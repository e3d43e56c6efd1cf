// Weight gradients for m = 64 (n = 4096), bf16 inputs, fp32 gradients:
//     dR[k][j][i] = sum_t du[t][k][j] x[t][k*64+i]          dL[j][l][k] = sum_t dy[t][l*64+j] u[t][k][j]
// (the chain rule through y = P L P^T R x with u = P^T R x kept per block, du = L^T applied to P dy).
//
// Every block's gradient is a 64 x 64 GEMM whose reduction dimension is the TOKEN index, so both operands
// are read "MN-major" (tokens along K).  The two intermediates come from the first stage of the fused
// forward kernel (u, in its exchange layout [tile][j][k/8][t%64][k%8]) and from the first stage of the
// fused backward kernel (du as [tile][k][j/8][t%64][j%8], and the transposed dy it builds anyway as
// [tile][j][l/8][t%64][l%8]); each 8 KB run of those buffers is at once an A or B operand of 64 tokens for
// tcgen05.mma - 8 x 8 core matrices of eight consecutive tokens by eight consecutive rows.  x itself is used
// straight from its natural layout (64 x 64 boxes, 128B swizzle).
//
// One CTA owns 16 blocks of one gradient - their 16 accumulators of 64 x 64 fp32 fill TMEM exactly (two
// M = 64 accumulators share each 32-lane quarter) - and a slice of the token tiles; it runs 64 MMAs per
// tile and never leaves TMEM until its tiles are done, then adds its partial sums to the output with
// vector reductions in L2.  Summation order across CTAs is not fixed, so results can differ in the last
// fp32 bits from run to run.
#include <cstdlib>

#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

constexpr int kN = 4096;
constexpr int kEpiWarps = 8, kLoadWarp0 = 8, kMmaWarp = 12;
constexpr int kThreads = 13 * 32;
constexpr int kSlotBytes = 16384;                  // A operand + B operand of one block, 64 tokens
constexpr int kSlots = 12, kQuads = 3;
constexpr int kSmemBytes = kSlots * kSlotBytes + 1024;

struct DwParams {
    const __nv_bfloat16 *u;      // [tiles][64 j][8][64][8]
    const __nv_bfloat16 *du;     // [tiles][64 k][8][64][8]
    const __nv_bfloat16 *dyp;    // [tiles][64 j][8][64][8]
    float *dL, *dR;
    unsigned *status;
    int tiles;
    int slices;                  // CTAs per block group; CTA s takes tiles s, s + slices, ...
};

__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}
__device__ __forceinline__ bool wait_fast(uint32_t bar, uint32_t parity, unsigned *status, volatile int *dead,
                                          unsigned code)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait(bar, parity, status, dead, code);
}
__device__ __forceinline__ void red_add_v4(float *p, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(__uint_as_float(a)),
                 "f"(__uint_as_float(b)), "f"(__uint_as_float(c)), "f"(__uint_as_float(d))
                 : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
fused_bwd_dw_m64_kernel(const __grid_constant__ CUtensorMap tm_x, const DwParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kQuads], bar_empty[kQuads], bar_acc;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead;

    const uint32_t ring0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = (int)blockIdx.x & 7, first = (int)blockIdx.x >> 3, step = p.slices;
    const bool is_R = grp < 4;
    const int blk0 = (grp & 3) * 16;

    if (threadIdx.x == 0) {
        for (int q = 0; q < kQuads; ++q) {
            mbar_init(smem_u32(&bar_full[q]), 4);
            mbar_init(smem_u32(&bar_empty[q]), 1);
        }
        mbar_init(smem_u32(&bar_acc), 1);
        fence_mbar_init();
        dead = 0;
        tma_prefetch_desc(&tm_x);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    const uint32_t full0 = smem_u32(bar_full), empty0 = smem_u32(bar_empty), acc = smem_u32(&bar_acc);

    if (first < p.tiles) {
        if (warp >= kLoadWarp0 && warp < kLoadWarp0 + 4) {
            if (lane == 0) {
                // loader pw fetches slot pw of every group of four: block blk0 + 4q + pw
                const int pw = warp - kLoadWarp0;
                int g = 0;
                uint32_t ph = 0;
                for (int tile = first; tile < p.tiles; tile += step) {
#pragma unroll 1
                    for (int q = 0; q < 4; ++q) {
                        const int blk = blk0 + q * 4 + pw;
                        if (!wait_fast(empty0 + g * 8, ph ^ 1, p.status, &dead, kErrSlotWait)) break;
                        const uint32_t slot = ring0 + (g * 4 + pw) * kSlotBytes;
                        const long long run = ((long long)tile * 64 + blk) * 4096;
                        mbar_expect_tx(full0 + g * 8, kSlotBytes);
                        if (is_R) {
                            bulk_load(slot, p.du + run, 8192, full0 + g * 8);
                            tma_load_2d(slot + 8192, &tm_x, blk * 64, tile * 64, full0 + g * 8);
                        } else {
                            bulk_load(slot, p.dyp + run, 8192, full0 + g * 8);
                            bulk_load(slot + 8192, p.u + run, 8192, full0 + g * 8);
                        }
                        if (++g == kQuads) { g = 0; ph ^= 1; }
                    }
                    if (dead) break;
                }
            }
        } else if (warp == kMmaWarp) {
            if (lane == 0) {
                constexpr uint32_t idesc = make_idesc_bf16(64, 64, 1, 1);      // both operands token-major
                // 8 x 8 core matrices: 128 B apart along tokens (K), 1 KB apart along rows (M / N)
                const uint64_t d_run = make_smem_desc(0, 128, 1024, 0);
                const uint64_t d_x = make_smem_desc(0, 16, 1024, kSwizzle128);
                const uint64_t a_base = d_run | (uint64_t)(ring0 >> 4);
                const uint64_t b_base = (is_R ? d_x : d_run) | (uint64_t)((ring0 + 8192) >> 4);
                const uint32_t kstep_b = is_R ? 128 : 16;                        // 16 tokens: 2 KB of x rows, or 2 core rows
                int g = 0;
                uint32_t ph = 0;
                bool ok = true;
                for (int tile = first; ok && tile < p.tiles; tile += step) {
                    const uint32_t acc_flag = tile != first;
#pragma unroll 1
                    for (int q = 0; q < 4; ++q) {
                        if (!wait_fast(full0 + g * 8, ph, p.status, &dead, kErrTmaWait)) { ok = false; break; }
                        tc_fence_after();
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int b = q * 4 + i;
                            const uint32_t d = tmem_base + ((uint32_t)((b >> 3) * 16) << 16) + (b & 7) * 64;
                            const uint64_t ad = a_base + (uint64_t)((g * 4 + i) * (kSlotBytes >> 4));
                            const uint64_t bd = b_base + (uint64_t)((g * 4 + i) * (kSlotBytes >> 4));
                            mma_f16_ss(d, ad, bd, idesc, acc_flag);
                            mma_f16_ss(d, ad + 16, bd + kstep_b, idesc, 1);
                            mma_f16_ss(d, ad + 32, bd + 2 * kstep_b, idesc, 1);
                            mma_f16_ss(d, ad + 48, bd + 3 * kstep_b, idesc, 1);
                        }
                        mma_commit(empty0 + g * 8);
                        if (++g == kQuads) { g = 0; ph ^= 1; }
                    }
                }
                if (ok) mma_commit(acc);
            }
        } else if (warp < kEpiWarps) {
            // partial sums -> gradient: lane i holds row 16 q4 + i%16 of block i/16 * 8 + b
            const int q4 = warp & 3, sub = warp >> 2;
            if (mbar_wait(acc, 0, p.status, &dead, kErrMmaWait)) {
                tc_fence_after();
                const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16);
                const int row = q4 * 16 + (lane & 15);
                float *out = (is_R ? p.dR : p.dL) + (long long)(blk0 + (lane >> 4) * 8) * 4096 + row * 64;
#pragma unroll 1
                for (int b = sub * 4; b < sub * 4 + 4; ++b) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint32_t v[2][16];
                        tmem_ld16(lane_base + b * 64 + h * 32, v[0]);
                        tmem_ld16(lane_base + b * 64 + h * 32 + 16, v[1]);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const uint32_t *w = &v[e >> 2][(e & 3) * 4];
                            red_add_v4(out + b * 4096 + h * 32 + e * 4, w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

}  // namespace
}  // namespace tc

constexpr size_t kDwCounterBytes = 65536;

// Workspace: [status 256 B][reserved 64 KB][u][du][P dy], each tokens (rounded up to 64) x 4096 bf16.
size_t fused_bwd_dw_m64_workspace_bytes(int64_t tokens, bool fixed_order)
{
    const size_t tiles = (size_t)((tokens + 63) / 64);
    return MONARCH_STATUS_BYTES + kDwCounterBytes + 3 * ((tiles * 64 * (size_t)tc::kN * 2 + 255) & ~(size_t)255) +
           (fixed_order ? kBwdPartialBytes : 0);
}

namespace {
// dL, dR += token reduction over the three intermediates
int launch_dw(const void *x, const void *u, const void *du, const void *dyp, float *dL, float *dR,
              unsigned *status, int64_t tokens, cudaStream_t s)
{
    using namespace tc;
    const long long tiles = (tokens + 63) / 64;
    CUtensorMap tm_x;
    MONARCH_TRY(encode_tmap_2d(&tm_x, x, (uint64_t)tokens, kN, kN * 2, 64, 64, 128));
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(fused_bwd_dw_m64_kernel,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    DwParams p;
    p.u = (const __nv_bfloat16 *)u;
    p.du = (const __nv_bfloat16 *)du;
    p.dyp = (const __nv_bfloat16 *)dyp;
    p.dL = dL;
    p.dR = dR;
    p.status = status;
    p.tiles = (int)tiles;
    int slices = sms / 8;
    if (slices < 1) slices = 1;
    if (slices > tiles) slices = (int)tiles;
    p.slices = slices;
    fused_bwd_dw_m64_kernel<<<8 * slices, kThreads, kSmemBytes, s>>>(tm_x, p);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

size_t exchange_bytes(int64_t tokens)
{
    const size_t tiles = (size_t)((tokens + 63) / 64);
    return (tiles * 64 * (size_t)tc::kN * 2 + 255) & ~(size_t)255;
}

int zero_grads(float *dL, float *dR, cudaStream_t s)
{
    const size_t gbytes = (size_t)tc::kN * 64 * sizeof(float);
    MONARCH_CUDA_TRY(cudaMemsetAsync(dL, 0, gbytes, s));
    MONARCH_CUDA_TRY(cudaMemsetAsync(dR, 0, gbytes, s));
    return MONARCH_OK;
}
}  // namespace

int fused_bwd_dw_m64(const void *x, const void *dy, const void *L, const void *R, float *dL, float *dR,
                     int accumulate, int64_t tokens, void *ws, cudaStream_t s, bool fixed_order)
{
    if (!accumulate && (!fixed_order || tokens == 0)) MONARCH_TRY(zero_grads(dL, dR, s));
    if (tokens == 0) return MONARCH_OK;
    const size_t ex = exchange_bytes(tokens);
    unsigned *status = (unsigned *)ws;
    char *u = (char *)ws + MONARCH_STATUS_BYTES + kDwCounterBytes;
    char *du = u + ex, *dyp = du + ex;
    MONARCH_TRY(fused_fwd_m64_stage1(x, R, u, tokens, status, s));
    if (fixed_order)
        return fused_bwd_all_m64(x, dy, L, R, u, nullptr, du, dyp, dL, dR, (unsigned *)((char *)ws + MONARCH_STATUS_BYTES), status,
                                 tokens, s, (float *)(dyp + ex), accumulate);
    // the one-launch backward with its dx part switched off: du and P dy are consumed from L2 as they appear
    // instead of after a launch of their own (it declines, before launching anything, on a GPU too small to hold
    // all of its CTAs at once; then the three-launch form below runs)
    unsigned *counters = (unsigned *)((char *)ws + MONARCH_STATUS_BYTES);
    const int rc = fused_bwd_all_m64(x, dy, L, R, u, nullptr, du, dyp, dL, dR, counters, status, tokens, s);
    if (rc != MONARCH_ERR_UNSUPPORTED) return rc;
    MONARCH_TRY(fused_bwd_m64_stage1(dy, L, du, dyp, tokens, status, s));
    return launch_dw(x, u, du, dyp, dL, dR, status, tokens, s);
}

// Workspace: [status 256 B][tile counters 64 KB][du][P dy][u], each tokens (rounded up to 64) x 4096 bf16.
size_t fused_bwd_m64_workspace_bytes(int64_t tokens, bool fixed_order)
{
    return MONARCH_STATUS_BYTES + kDwCounterBytes + 3 * exchange_bytes(tokens) + (fixed_order ? kBwdPartialBytes : 0);
}

int fused_bwd_m64(const void *x, const void *dy, const void *L, const void *R, const void *u_saved,
                  void *dx, float *dL, float *dR, int accumulate, int64_t tokens, void *ws,
                  cudaStream_t s, bool fixed_order)
{
    if (!accumulate && (!fixed_order || tokens == 0)) MONARCH_TRY(zero_grads(dL, dR, s));
    if (tokens == 0) return MONARCH_OK;
    const size_t ex = exchange_bytes(tokens);
    unsigned *status = (unsigned *)ws;
    unsigned *counters = (unsigned *)((char *)ws + MONARCH_STATUS_BYTES);
    char *du = (char *)ws + MONARCH_STATUS_BYTES + kDwCounterBytes;
    char *dyp = du + ex, *u_own = dyp + ex;
    const void *u = u_saved;
    if (!u) {
        MONARCH_TRY(fused_fwd_m64_stage1(x, R, u_own, tokens, status, s));
        u = u_own;
    }
#ifdef MONARCH_TRACE
    // debug builds: the two-kernel form (backward kernel, then the token reduction), for comparison
    static const bool split = getenv("MONARCH_BWD_SPLIT") != nullptr;
    if (split) {
        MONARCH_TRY(fused_bwd_dx_m64_keep(dy, L, R, dx, du, dyp, counters, status, tokens, s));
        return launch_dw(x, u, du, dyp, dL, dR, status, tokens, s);
    }
#endif
    // the one-launch form declines, before launching anything, on a GPU too small to hold all of its CTAs at once
    // (or for more tiles than it has counters): then the backward kernel and the token reduction run as two launches
    if (fixed_order)
        return fused_bwd_all_m64(x, dy, L, R, u, dx, du, dyp, dL, dR, counters, status, tokens, s, (float *)(u_own + ex),
                                 accumulate);
    const int rc = fused_bwd_all_m64(x, dy, L, R, u, dx, du, dyp, dL, dR, counters, status, tokens, s);
    if (rc != MONARCH_ERR_UNSUPPORTED) return rc;
    MONARCH_TRY(fused_bwd_dx_m64_keep(dy, L, R, dx, du, dyp, counters, status, tokens, s));
    return launch_dw(x, u, du, dyp, dL, dR, status, tokens, s);
}

}  // namespace monarch
