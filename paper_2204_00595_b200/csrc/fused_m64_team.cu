// Fused forward y = P L P^T R x for m = 64 (n = 4096), bf16, "team" schedule.
//
// Same data flow as fused_m64.cu (stage 1 writes u' = P R x to an L2-resident exchange buffer in the operand
// layout of stage 2; Section 3.3 steps 1-3), but every CTA does BOTH stages: the eight CTAs of a team take the
// eight stage-1 block groups of a 64-token tile and, one tile later, its eight stage-2 groups.  No SM waits on
// another kind of SM, the single MMA-issuing thread of each CTA is busy all the time (S1(t+1), S2(t), S1(t+2),
// ...), and the tile whose u' is read back was written a few thousand cycles earlier by the same team.
//
// Shared memory: R group (64 KB) + L half-group (64 KB) resident, 4 staging buffers, an 8-slot operand ring.
// TMEM: stage-1 accumulators in columns [0,256) (blocks 0-3 / 4-7 in the two 16-lane halves of every quarter),
// stage-2 accumulators in columns [256,512) (blocks 0-7 / 8-15), each single-buffered: the other stage's MMAs
// run while an accumulator set is drained.
#include <cstdlib>

#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

constexpr int kM = 64;
constexpr int kN = kM * kM;
// warps: 0-7 epilogue (two halves of four), 8-9 operand loaders, 10 MMA, 11-12 store threads, 13 L2 prefetch
constexpr int kEpiWarps = 8, kLoadWarp0 = 8, kMmaWarp = 10, kStoreWarp0 = 11, kPrefetchWarp = 13;
constexpr int kThreads = 14 * 32;
constexpr int kRBytes = 65536, kLBytes = 65536;
constexpr int kStageBytes = 8192, kStagesPerHalf = 2;
constexpr int kSlotBytes = 8192, kPairs = 4;                   // ring of 8 slots, handed over in pairs
constexpr int kSmemBytes = kRBytes + kLBytes + 2 * kStagesPerHalf * kStageBytes + 2 * kPairs * kSlotBytes + 1024;
constexpr unsigned kS1Arrivals = 8 * 2;                        // 8 team members x 2 store threads per tile
constexpr unsigned kS2Groups = 8;

struct TeamParams {
    __nv_bfloat16 *u;          // exchange buffer, [tiles][64 j][8][64 t][8] bf16
    unsigned *counters;        // one per 64-token tile, zero between calls
    unsigned *status;
    const __nv_bfloat16 *x;    // input (for L2 prefetch hints only; the data path goes through TMA)
    long long tokens;
    const __nv_bfloat16 *bias; // optional [n]: added to the output (feed-forward block, Section 4)
    int gelu;                  // apply erf-GELU after the bias
    int tiles;
    int teams;                 // CTA team c takes tiles c, c + teams, ...
    long long *trace;          // optional per-CTA timeline (debug builds), else null
};

#ifdef MONARCH_TRACE
#define TTRACE(item, slot, val) do { if (p.trace && (item) < 16) p.trace[((size_t)blockIdx.x * 16 + (item)) * 8 + (slot)] = (val); } while (0)
#define TCLK() clock64()
#else
#define TTRACE(item, slot, val) do { } while (0)
#define TCLK() 0ll
#endif

struct Bars {
    uint64_t w;
    uint64_t full[kPairs], empty[kPairs];
    uint64_t s1_full, s1_empty, s2_full, s2_empty;
    uint64_t st_full[2 * kStagesPerHalf], st_free[2 * kStagesPerHalf];
};

__device__ __forceinline__ unsigned ld_acquire(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void fence_proxy_async_global()
{
    asm volatile("fence.proxy.async.global;" ::: "memory");
}
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

__global__ void __launch_bounds__(kThreads, 1)
fused_fwd_m64_team_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_R,
                          const __grid_constant__ CUtensorMap tm_L, const __grid_constant__ CUtensorMap tm_u,
                          const __grid_constant__ CUtensorMap tm_y, const TeamParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) Bars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead_s;
    __shared__ int dep_items_s;
    __shared__ __align__(16) __nv_bfloat16 bias_s[32 * 16];   // this CTA's slice of the bias: [l local][j local]

    [[maybe_unused]] const long long t_entry = TCLK();
    const uint32_t smemR = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t smemL = smemR + kRBytes;
    const uint32_t stage0 = smemL + kLBytes;
    const uint32_t ring0 = stage0 + 2 * kStagesPerHalf * kStageBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp = (int)blockIdx.x & 7, team = (int)blockIdx.x >> 3;
    const int hj = grp >> 1, hl = grp & 1;           // stage 2: 16 blocks j, 32 output rows l
    volatile int *dead = &dead_s;
    volatile int *dep_items = &dep_items_s;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars.w), 1);
        for (int g = 0; g < kPairs; ++g) {
            mbar_init(smem_u32(&bars.full[g]), 2);           // two loads, one per loader warp
            mbar_init(smem_u32(&bars.empty[g]), 1);
        }
        mbar_init(smem_u32(&bars.s1_full), 1);
        mbar_init(smem_u32(&bars.s1_empty), kEpiWarps);
        mbar_init(smem_u32(&bars.s2_full), 1);
        mbar_init(smem_u32(&bars.s2_empty), kEpiWarps);
        for (int k = 0; k < 2 * kStagesPerHalf; ++k) {
            mbar_init(smem_u32(&bars.st_full[k]), 4);        // the four warps of an epilogue half
            mbar_init(smem_u32(&bars.st_free[k]), 1);
        }
        fence_mbar_init();
        dead_s = 0;
        dep_items_s = 0;
        tma_prefetch_desc(&tm_x); tma_prefetch_desc(&tm_R); tma_prefetch_desc(&tm_L);
        tma_prefetch_desc(&tm_u); tma_prefetch_desc(&tm_y);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    if (p.bias != nullptr && threadIdx.x >= 64 && threadIdx.x < 128) {
        // global loads stay out of the steady state: they slow the MMA-issuing thread down
        const int l = (threadIdx.x - 64) >> 1, half = threadIdx.x & 1;
        *reinterpret_cast<uint4 *>(&bias_s[l * 16 + half * 8]) =
            __ldg(reinterpret_cast<const uint4 *>(p.bias + (hl * 32 + l) * kM + hj * 16 + half * 8));
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    if (threadIdx.x == 0) { TTRACE(15, 0, t_entry); TTRACE(15, 1, TCLK()); }

    // number of tiles of this team; step `it` does S1(tile it) then S2(tile it-1)
    const int nt = team < p.tiles ? (p.tiles - team + p.teams - 1) / p.teams : 0;
    const uint32_t full0 = smem_u32(bars.full), empty0 = smem_u32(bars.empty);
    const uint32_t s1f = smem_u32(&bars.s1_full), s1e = smem_u32(&bars.s1_empty);
    const uint32_t s2f = smem_u32(&bars.s2_full), s2e = smem_u32(&bars.s2_empty);

    if (nt > 0 && warp >= kLoadWarp0 && warp < kLoadWarp0 + 2) {
        // ------------------------------------------------------------ loaders: warp pw fills slot pw of every pair
        if (lane == 0) {
            const int pw = warp - kLoadWarp0;
            if (pw == 0) {
                const uint32_t wbar = smem_u32(&bars.w);
                mbar_expect_tx(wbar, kRBytes + kLBytes);
                for (int b = 0; b < 8; ++b) tma_load_2d(smemR + b * 8192, &tm_R, 0, (grp * 8 + b) * kM, wbar);
                for (int b = 0; b < 16; ++b)
                    tma_load_2d(smemL + b * 4096, &tm_L, 0, (hj * 16 + b) * kM + hl * 32, wbar);
            }
            uint32_t round = 0;                          // completed passes over the ring
            bool ok = true;
            for (int it = 0; ok && it <= nt; ++it) {
                if (it < nt) {
                    const int tile = team + it * p.teams;
#pragma unroll
                    for (int g = 0; g < kPairs; ++g) {
                        if (!wait_fast(empty0 + g * 8, (round & 1) ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
                        mbar_expect_tx(full0 + g * 8, kSlotBytes);
                        tma_load_2d(ring0 + (g * 2 + pw) * kSlotBytes, &tm_x, (grp * 8 + g * 2 + pw) * kM, tile * 64,
                                    full0 + g * 8);
                    }
                    ++round;
                }
                if (ok && it >= 1) {
                    const int tile = team + (it - 1) * p.teams;
                    if (pw == 0) {
                        // wait until the whole team has published its part of u' for this tile
                        const unsigned *ctr = p.counters + tile;
                        if (ld_acquire(ctr) < kS1Arrivals) {
                            const unsigned long long t0 = global_timer_ns();
                            while (ld_acquire(ctr) < kS1Arrivals) {
                                if (*dead || global_timer_ns() - t0 > kWaitLimitNs) {
                                    *dead = 1;
                                    atomicCAS(p.status, 0u, (unsigned)kErrPeerWait);
                                    ok = false;
                                    break;
                                }
                            }
                            if (!ok) break;
                        }
                        // the last team member to get here clears the counter for the next call
                        const unsigned old = atomicAdd(p.counters + tile, 1u);
                        if (old + 1 == kS1Arrivals + kS2Groups) atomicExch(p.counters + tile, 0u);
                        fence_proxy_async_global();
                        __threadfence_block();
                        *dep_items = it;                      // monotonic
                    } else {
                        if (*dep_items < it) {
                            const unsigned long long t0 = global_timer_ns();
                            while (*dep_items < it) {
                                if (*dead || global_timer_ns() - t0 > kWaitLimitNs) {
                                    *dead = 1;
                                    atomicCAS(p.status, 0u, (unsigned)kErrPeerWait);
                                    ok = false;
                                    break;
                                }
                            }
                            if (!ok) break;
                        }
                        __threadfence_block();
                        fence_proxy_async_global();
                    }
                    const __nv_bfloat16 *usrc = p.u + ((long long)tile * 64 + hj * 16 + pw) * 4096;
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {
#pragma unroll
                        for (int g = 0; g < kPairs; ++g) {
                            if (!wait_fast(empty0 + g * 8, (round & 1) ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
                            mbar_expect_tx(full0 + g * 8, kSlotBytes);
                            bulk_load(ring0 + (g * 2 + pw) * kSlotBytes, usrc + (size_t)(rr * 8 + g * 2) * 4096, 8192,
                                      full0 + g * 8);
                        }
                        if (!ok) break;
                        ++round;
                    }
                }
            }
        }
    } else if (nt > 0 && warp == kMmaWarp) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && mbar_wait(smem_u32(&bars.w), 0, p.status, dead, kErrTmaWait)) {
            tc_fence_after();
            const uint64_t a_x = make_smem_desc(0, 16, 1024, kSwizzle128) | (uint64_t)(ring0 >> 4);
            const uint64_t a_u = make_smem_desc(0, 1024, 128, 0) | (uint64_t)(ring0 >> 4);
            const uint64_t b_R = make_smem_desc(0, 16, 1024, kSwizzle128) | (uint64_t)(smemR >> 4);
            const uint64_t b_L = make_smem_desc(0, 16, 1024, kSwizzle128) | (uint64_t)(smemL >> 4);
            constexpr uint32_t idesc1 = make_idesc_bf16(64, 64, 0, 0), idesc2 = make_idesc_bf16(64, 32, 0, 0);
            uint32_t round = 0;
            bool ok = true;
            for (int it = 0; ok && it <= nt; ++it) {
                if (it < nt) {
                    TTRACE(it, 0, TCLK());
                    if (!wait_fast(s1e, (it & 1) ^ 1, p.status, dead, kErrTmemWait)) break;
                    tc_fence_after();
                    TTRACE(it, 1, TCLK());
                    [[maybe_unused]] long long wsum = 0;
#pragma unroll
                    for (int g = 0; g < kPairs; ++g) {
                        [[maybe_unused]] const long long c0 = TCLK();
                        if (!wait_fast(full0 + g * 8, round & 1, p.status, dead, kErrTmaWait)) { ok = false; break; }
                        tc_fence_after();
                        wsum += TCLK() - c0;
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            const int b = g * 2 + i;
                            const uint64_t ad = a_x + (uint64_t)(b * (kSlotBytes >> 4));
                            const uint64_t bd = b_R + b * 512;
                            const uint32_t d = tmem_base + ((uint32_t)((b >> 2) * 16) << 16) + (b & 3) * 64;
                            mma_f16_ss(d, ad, bd, idesc1, 0);
                            mma_f16_ss(d, ad + 2, bd + 2, idesc1, 1);
                            mma_f16_ss(d, ad + 4, bd + 4, idesc1, 1);
                            mma_f16_ss(d, ad + 6, bd + 6, idesc1, 1);
                        }
                        mma_commit(empty0 + g * 8);
                    }
                    if (!ok) break;
                    mma_commit(s1f);
                    ++round;
                    TTRACE(it, 2, wsum);
                    TTRACE(it, 3, TCLK());
                }
                if (it >= 1) {
                    if (!wait_fast(s2e, ((it - 1) & 1) ^ 1, p.status, dead, kErrTmemWait)) break;
                    tc_fence_after();
                    TTRACE(it - 1, 4, TCLK());
                    [[maybe_unused]] long long wsum2 = 0;
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {
#pragma unroll
                        for (int g = 0; g < kPairs; ++g) {
                            [[maybe_unused]] const long long c0 = TCLK();
                            if (!wait_fast(full0 + g * 8, round & 1, p.status, dead, kErrTmaWait)) { ok = false; break; }
                            tc_fence_after();
                            wsum2 += TCLK() - c0;
#pragma unroll
                            for (int i = 0; i < 2; ++i) {
                                const int b = rr * 8 + g * 2 + i;
                                const uint64_t ad = a_u + (uint64_t)((g * 2 + i) * (kSlotBytes >> 4));
                                const uint64_t bd = b_L + b * 256;
                                const uint32_t d = tmem_base + ((uint32_t)((b >> 3) * 16) << 16) + 256 + (b & 7) * 32;
                                mma_f16_ss(d, ad, bd, idesc2, 0);
                                mma_f16_ss(d, ad + 128, bd + 2, idesc2, 1);
                                mma_f16_ss(d, ad + 256, bd + 4, idesc2, 1);
                                mma_f16_ss(d, ad + 384, bd + 6, idesc2, 1);
                            }
                            mma_commit(empty0 + g * 8);
                        }
                        if (!ok) break;
                        ++round;
                    }
                    if (!ok) break;
                    mma_commit(s2f);
                    TTRACE(it - 1, 5, wsum2);
                    TTRACE(it - 1, 6, TCLK());
                }
            }
        }
    } else if (nt > 0 && warp < kEpiWarps) {
        // ------------------------------------------------------------ epilogue: TMEM -> bf16 -> staging
        const int q4 = warp & 3, sub = warp >> 2, h = lane >> 4;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16);
        const int row = q4 * 16 + (lane & 15);
        const uint32_t my_stage = stage0 + sub * kStagesPerHalf * kStageBytes;
        const uint32_t stf0 = smem_u32(bars.st_full) + sub * kStagesPerHalf * 8;
        const uint32_t stfree0 = smem_u32(bars.st_free) + sub * kStagesPerHalf * 8;
        uint32_t nchunk = 0;
        bool ok = true;
        for (int it = 0; ok && it <= nt; ++it) {
            if (it < nt) {
                if (!wait_fast(s1f, it & 1, p.status, dead, kErrMmaWait)) break;
                tc_fence_after();
#pragma unroll 1
                for (int c = sub; c < 8; c += 2, ++nchunk) {
                    const uint32_t k = nchunk & (kStagesPerHalf - 1);
                    const uint32_t sbuf = my_stage + k * kStageBytes;
                    // chunk = 8 consecutive j; this lane holds blocks 4h..4h+3 of row `row`
                    uint32_t v[4][8];
#pragma unroll
                    for (int kb = 0; kb < 4; ++kb) tmem_ld8(lane_base + kb * 64 + c * 8, v[kb]);
                    tmem_ld_wait();
                    if (c + 2 >= 8) {
                        // the accumulators are in registers: hand them back before waiting for a staging buffer
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(s1e);
                    }
                    if (!wait_fast(stfree0 + k * 8, ((nchunk / kStagesPerHalf) & 1) ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const uint32_t o0 = pack_bf16(__uint_as_float(v[0][q]), __uint_as_float(v[1][q]));
                        const uint32_t o1 = pack_bf16(__uint_as_float(v[2][q]), __uint_as_float(v[3][q]));
                        // staging [j local 8][t 64][8 k]: the 1 KB slab of u'[tile][j][k/8 = grp]
                        asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(sbuf + q * 1024 + row * 16 + h * 8), "r"(o0), "r"(o1) : "memory");
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(stf0 + k * 8);
                }
            }
            if (ok && it >= 1) {
                if (!wait_fast(s2f, (it - 1) & 1, p.status, dead, kErrMmaWait)) break;
                tc_fence_after();
#pragma unroll 1
                for (int c = sub; c < 8; c += 2, ++nchunk) {
                    const uint32_t k = nchunk & (kStagesPerHalf - 1);
                    const uint32_t sbuf = my_stage + k * kStageBytes;
                    // chunk = 4 consecutive output rows l; lanes i and i+16 hold blocks 0-7 and 8-15
                    uint32_t v[8][4];
#pragma unroll
                    for (int a = 0; a < 8; ++a) tmem_ld4(lane_base + 256 + a * 32 + c * 4, v[a]);
                    tmem_ld_wait();
                    if (c + 2 >= 8) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(s2e);
                    }
                    if (!wait_fast(stfree0 + k * 8, ((nchunk / kStagesPerHalf) & 1) ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
                    if (p.bias != nullptr) {
                        // output element (l, j): l = 32 hl + 4c + q, j = 16 hj + 8h + a
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const uint4 bq = *reinterpret_cast<const uint4 *>(&bias_s[(c * 4 + q) * 16 + h * 8]);
                            const uint32_t bw[4] = {bq.x, bq.y, bq.z, bq.w};
#pragma unroll
                            for (int a = 0; a < 8; ++a) {
                                const float b = __uint_as_float((a & 1) ? (bw[a >> 1] & 0xFFFF0000u) : (bw[a >> 1] << 16));
                                float f = __uint_as_float(v[a][q]) + b;
                                if (p.gelu) f = gelu_fast(f);
                                v[a][q] = __float_as_uint(f);
                            }
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint32_t o0 = pack_bf16(__uint_as_float(v[0][q]), __uint_as_float(v[1][q]));
                        const uint32_t o1 = pack_bf16(__uint_as_float(v[2][q]), __uint_as_float(v[3][q]));
                        const uint32_t o2 = pack_bf16(__uint_as_float(v[4][q]), __uint_as_float(v[5][q]));
                        const uint32_t o3 = pack_bf16(__uint_as_float(v[6][q]), __uint_as_float(v[7][q]));
                        // staging [l local 4][t 64][16 j]
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sbuf + q * 2048 + row * 32 + h * 16),
                                     "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(stf0 + k * 8);
                }
            }
        }
    } else if (nt > 0 && warp >= kStoreWarp0 && warp < kStoreWarp0 + 2) {
        // ------------------------------------------------------------ store threads (one per epilogue half)
        if (lane == 0) {
            const int sub = warp - kStoreWarp0;
            const uint32_t my_stage = stage0 + sub * kStagesPerHalf * kStageBytes;
            const uint32_t stf0 = smem_u32(bars.st_full) + sub * kStagesPerHalf * 8;
            const uint32_t stfree0 = smem_u32(bars.st_free) + sub * kStagesPerHalf * 8;
            uint32_t nchunk = 0;
            int unfreed = -1;                              // staging buffer whose store may still be reading
            bool ok = true;
            for (int it = 0; ok && it <= nt; ++it) {
                if (it < nt) {
                    const int tile = team + it * p.teams;
#pragma unroll 1
                    for (int c = sub; c < 8; c += 2, ++nchunk) {
                        const uint32_t k = nchunk & (kStagesPerHalf - 1);
                        if (!wait_fast(stf0 + k * 8, (nchunk / kStagesPerHalf) & 1, p.status, dead, kErrMmaWait)) { ok = false; break; }
                        // u' as 8-byte words: [tile*64 + j][k/8][128 words]; 8 rows (j) of 1 KB
                        asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(&tm_u),
                                     "r"(my_stage + k * kStageBytes), "r"(0), "r"(grp), "r"(tile * 64 + c * 8) : "memory");
                        tma_store_commit();
                        if (unfreed >= 0) {
                            tma_store_wait_read<1>();
                            mbar_arrive(stfree0 + unfreed * 8);
                        }
                        unfreed = (int)k;
                    }
                    if (!ok) break;
                    // this member's part of u'[tile] is complete: publish it (nothing else to store meanwhile -
                    // the stage-2 epilogue of the previous tile starts a few thousand cycles later)
                    tma_store_wait_all<0>();
                    if (unfreed >= 0) { mbar_arrive(stfree0 + unfreed * 8); unfreed = -1; }
                    fence_proxy_async_global();
                    __threadfence();
                    atomicAdd(p.counters + tile, 1u);
                }
                if (it >= 1) {
                    const int tile = team + (it - 1) * p.teams;
#pragma unroll 1
                    for (int c = sub; c < 8; c += 2, ++nchunk) {
                        const uint32_t k = nchunk & (kStagesPerHalf - 1);
                        if (!wait_fast(stf0 + k * 8, (nchunk / kStagesPerHalf) & 1, p.status, dead, kErrMmaWait)) { ok = false; break; }
                        // y as [l][t][j]: box 16 j x 64 t x 4 l; rows past the last token are clipped
                        asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(&tm_y),
                                     "r"(my_stage + k * kStageBytes), "r"(hj * 16), "r"(tile * 64), "r"(hl * 32 + c * 4) : "memory");
                        tma_store_commit();
                        if (unfreed >= 0) {
                            tma_store_wait_read<1>();
                            mbar_arrive(stfree0 + unfreed * 8);
                        }
                        unfreed = (int)k;
                    }
                }
            }
            tma_store_wait_all<0>();
        }
    }

    else if (nt > 0 && warp == kPrefetchWarp) {
        // ------------------------------------------------------------ L2 prefetch hints for the next x tiles
        // The operand ring holds less than one tile, so an x tile is requested only ~2 k cycles before the MMAs
        // want it - less than a trip to DRAM.  One tile ahead, ask L2 for this CTA's 8 KB row segments.
        for (int it = 0; it + 1 < nt; ++it) {
            const int tile = team + (it + 1) * p.teams;
            const char *base = reinterpret_cast<const char *>(p.x) + ((long long)tile * 64 * kN + grp * 8 * kM) * 2;
#pragma unroll 1
            for (int i = 0; i < 16; ++i) {
                const int t = i * 4 + (lane >> 3);
                if ((long long)tile * 64 + t < p.tokens)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(base + (long long)t * (kN * 2) + (lane & 7) * 128));
            }
            // pace: one tile of hints per tile of stage-1 MMAs
            if (!wait_fast(s1f, it & 1, p.status, dead, kErrMmaWait)) break;
        }
    }

    if (threadIdx.x == 0) TTRACE(15, 2, TCLK());
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) TTRACE(15, 3, TCLK());
    if (warp == 0) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0) TTRACE(15, 4, TCLK());
}

}  // namespace
}  // namespace tc

namespace {
constexpr size_t kTeamCounterBytes = 65536;

int launch_team(const void *x, const void *L, const void *R, const void *bias, int gelu, void *y, void *u,
                unsigned *counters, unsigned *status, int64_t tokens, cudaStream_t s)
{
    using namespace tc;
    const long long tiles = (tokens + 63) / 64;
    if (tiles * 4 > (long long)kTeamCounterBytes) return MONARCH_ERR_UNSUPPORTED;
    CUtensorMap tm_x, tm_R, tm_L, tm_u, tm_y;
    MONARCH_TRY(encode_tmap_2d(&tm_x, x, (uint64_t)tokens, kN, kN * 2, 64, 64, 128));
    MONARCH_TRY(encode_tmap_2d(&tm_R, R, kN, kM, kM * 2, 64, 64, 128));
    MONARCH_TRY(encode_tmap_2d(&tm_L, L, kN, kM, kM * 2, 32, 64, 128));
    {
        const uint64_t dims[3] = {128, 8, (uint64_t)tiles * 64}, strides[2] = {1024, 8192};
        const uint32_t box[3] = {128, 1, 8};
        MONARCH_TRY(encode_tmap_nd(&tm_u, u, 8, 3, dims, strides, box));
        const uint64_t ydims[3] = {64, (uint64_t)tokens, 64}, ystrides[2] = {(uint64_t)kN * 2, 128};
        const uint32_t ybox[3] = {16, 64, 4};
        MONARCH_TRY(encode_tmap_nd(&tm_y, y, 2, 3, ydims, ystrides, ybox));
    }
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(fused_fwd_m64_team_kernel,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    TeamParams p;
    p.status = status;
    p.counters = counters;
    p.u = (__nv_bfloat16 *)u;
    p.x = (const __nv_bfloat16 *)x;
    p.tokens = tokens;
    p.bias = (const __nv_bfloat16 *)bias;
    p.gelu = gelu;
    p.tiles = (int)tiles;
    int teams = sms / 8;
    if (teams < 1) teams = 1;
    if (teams > tiles) teams = (int)tiles;
    p.teams = teams;
    p.trace = nullptr;
#ifdef MONARCH_TRACE
    if (const char *e = getenv("MONARCH_TRACE_PTR")) p.trace = (long long *)strtoull(e, nullptr, 0);
#endif
    fused_fwd_m64_team_kernel<<<8 * teams, kThreads, kSmemBytes, s>>>(tm_x, tm_R, tm_L, tm_u, tm_y, p);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

size_t exchange_bytes(int64_t tokens)
{
    const size_t tiles = (size_t)((tokens + 63) / 64);
    return (tiles * 64 * (size_t)tc::kN * 2 + 255) & ~(size_t)255;
}
}  // namespace

// Same workspace layout as the split schedule: [status 256 B][tile counters 64 KB][u'].
int fused_fwd_m64_team(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws,
                       cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    return launch_team(x, L, R, nullptr, 0, y, (char *)ws + MONARCH_STATUS_BYTES + kTeamCounterBytes,
                       (unsigned *)((char *)ws + MONARCH_STATUS_BYTES), (unsigned *)ws, tokens, s);
}

// One pass with the bias (and optionally GELU) applied in the stage-2 epilogue: y = act(M x + bias).
int fused_fwd_bias_m64(const void *x, const void *L, const void *R, const void *bias, int gelu, void *y,
                       int64_t tokens, void *ws, cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    return launch_team(x, L, R, bias, gelu, y, (char *)ws + MONARCH_STATUS_BYTES + kTeamCounterBytes,
                       (unsigned *)((char *)ws + MONARCH_STATUS_BYTES), (unsigned *)ws, tokens, s);
}

// Feed-forward block y = M2 GELU(M1 x + b1) + b2 as two passes of the same kernel; the hidden activations h
// (bf16) live in the workspace: [status][counters][u'][h].
size_t fused_mlp_fwd_m64_workspace_bytes(int64_t tokens)
{
    return MONARCH_STATUS_BYTES + kTeamCounterBytes + exchange_bytes(tokens) +
           (((size_t)tokens * tc::kN * 2 + 255) & ~(size_t)255);
}

int fused_mlp_fwd_m64(const void *x, const void *L1, const void *R1, const void *b1, const void *L2,
                      const void *R2, const void *b2, void *y, int64_t tokens, void *ws, cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    unsigned *status = (unsigned *)ws;
    unsigned *counters = (unsigned *)((char *)ws + MONARCH_STATUS_BYTES);
    char *u = (char *)ws + MONARCH_STATUS_BYTES + kTeamCounterBytes;
    char *h = u + exchange_bytes(tokens);
    MONARCH_TRY(launch_team(x, L1, R1, b1, 1, h, u, counters, status, tokens, s));
    return launch_team(h, L2, R2, b2, 0, y, u, counters, status, tokens, s);
}

}  // namespace monarch
