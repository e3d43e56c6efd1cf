// Fused Monarch forward for m = 64 (n = 4096), bf16 in/out, fp32 accumulation in TMEM: the SPLIT schedule.
// (The forward call itself uses the team schedule of fused_m64_team.cu, where every CTA does both stages; this
// kernel serves the stage-1-only launch inside monarch_bwd_dw, and debug builds can select it for comparison.)
//
// One persistent launch runs both block-diagonal stages and both permutations; the
// intermediate u never leaves the chip's L2.  CTAs (one per SM) specialise; both kinds work on
// 64-token tiles with tcgen05.mma M = 64, whose accumulators occupy one 16-lane half of every
// TMEM sub-partition, and both keep two tiles in flight so that one is drained while the next is
// multiplied:
//
//   S1 CTAs (8 groups g of `a` CTAs): keep the 8 blocks R_{8g..8g+7} resident in shared memory.
//       Per tile, TMA brings x[64 x 64] per block into a 128B-swizzled K-major ring slot;
//       4 MMAs (N = 64, K = 16) accumulate u[t][k][:] in TMEM columns [64*kb, 64*kb+64) of lane half
//       (tile parity).  With all 8 accumulators resident, the thread that owns token t picks
//       entry j of each block - a register renaming - and packs the 16 bytes u'[t][j][8g..8g+8)
//       of the exchange buffer, whose layout [tile][j][k/8][t%64][k%8] is the canonical no-swizzle
//       K-major operand layout of stage 2: the inner permutation P^T costs no data movement at all.
//   S2 CTAs (4 x 2 groups (hj, hl) of `b` CTAs): keep rows [32hl, 32hl+32) of L_{16hj..16hj+15}
//       resident.  One 8 KB bulk copy per block fetches u'_j[64 x 64] from L2; 4 MMAs (N = 32)
//       accumulate w[t][j][32hl..]; blocks 0-7 sit in lane half 0 and blocks 8-15 in lane half 1
//       of 256 TMEM columns (tile parity picks which 256).  Lanes i and i+16 of a warp then hold
//       blocks j0..j0+7 and j0+8..j0+15 of the same token and together form the 32 contiguous
//       bytes y[t][l*64 + 16hj .. 16hj+16): whole 32-byte sectors, which is what HBM writes need
//       (16-byte pieces were measured 5x slower).
//
// An S2 tile waits (bounded) on a per-tile counter that the S1 epilogues bump after their stores;
// S1 tiles wait on nothing, so the schedule cannot deadlock.  Warps 0-7 drain TMEM (two per
// sub-partition) into shared-memory staging buffers, warps 13-14 send those out with TMA tensor
// stores, warps 8-11 issue TMA/bulk loads, warp 12 issues every MMA.  The single-thread
// roles are latency-bound (one thread sustains about 50 GB/s of TMA issue and one MMA per
// 50-70 cycles), so loads are shared by four warps, ring slots are handled in groups of four (one
// full and one empty barrier per group), and the role loops are unrolled with static offsets.
#include <cstdlib>

#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

constexpr int kM = 64;
constexpr int kN = kM * kM;
constexpr int kEpiWarps = 8, kProdWarps = 4, kStoreWarps = 2;
constexpr int kMmaWarp = kEpiWarps + kProdWarps, kStoreWarp0 = kMmaWarp + 1;
constexpr int kThreads = (kEpiWarps + kProdWarps + 1 + kStoreWarps) * 32;
constexpr int kSlotBytes = 8192;                       // one [64 x 64] bf16 operand tile
constexpr int kSlots = 12, kQuads = kSlots / 4;        // ring, released and filled in groups of 4
constexpr int kWBytes = 65536;                         // resident weights: 8 R blocks, or 16 half L blocks
constexpr int kStageBytes = 8192, kStagesPerHalf = 4;  // output staging ring of each epilogue half
constexpr int kStages = 2 * kStagesPerHalf;
constexpr int kSmemBytes = kWBytes + kStages * kStageBytes + kSlots * kSlotBytes + 1024;
constexpr unsigned kS1Arrivals = 8 * 2;                // 8 S1 groups x 2 epilogue halves per tile
constexpr unsigned kS2Groups = 8;

struct FwdParams {
    __nv_bfloat16 *u;          // exchange buffer, [tiles][64 j][8][64 t][8] bf16
    __nv_bfloat16 *y;
    unsigned *counters;        // one per 64-token tile, zero between calls
    unsigned *status;
    long long tokens;
    int tiles;                 // 64-token tiles
    int a, b;                  // S1 CTAs per R group, S2 CTAs per L group
    long long *trace;          // optional per-CTA timeline (debug builds), else null
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
#ifdef MONARCH_TRACE
#define TRACE(slot) do { if (p.trace && nitem_t < 16) p.trace[((size_t)blockIdx.x * 16 + nitem_t) * 8 + (slot)] = clock64(); } while (0)
#else
#define TRACE(slot) do { } while (0)
#endif

// One try before the bounded wait: the common case in the single-thread role loops, where every
// extra dependent instruction costs several cycles.
__device__ __forceinline__ bool wait_fast(uint32_t bar, uint32_t parity, unsigned *status, volatile int *dead,
                                          unsigned code)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait(bar, parity, status, dead, code);
}

// Position of a tile's first block in the ring, in slot groups of four; advances without division.
template <int QUADS_PER_TILE> struct RingBase {
    int quad = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void next_tile()
    {
        quad += QUADS_PER_TILE;
#pragma unroll
        for (int i = 0; i < (QUADS_PER_TILE + kQuads - 1) / kQuads; ++i)
            if (quad >= kQuads) { quad -= kQuads; phase ^= 1; }
    }
    // group index and phase of the tile's q-th group
    __device__ __forceinline__ void at(int q, int &g, uint32_t &ph) const
    {
        g = quad + q;
        ph = phase;
#pragma unroll
        for (int i = 0; i < (QUADS_PER_TILE + kQuads - 1) / kQuads; ++i)
            if (g >= kQuads) { g -= kQuads; ph ^= 1; }
    }
};

template <bool S1>
__device__ __forceinline__ void role_body(const CUtensorMap &tm_x, const CUtensorMap &tm_R, const CUtensorMap &tm_L,
                                          const CUtensorMap &tm_u, const CUtensorMap &tm_y, const FwdParams &p, uint32_t smem0, uint64_t *bar_full, uint64_t *bar_empty,
                                          uint64_t *bar_acc_full, uint64_t *bar_acc_empty, uint64_t *bar_w,
                                          uint64_t *bar_st_full, uint64_t *bar_st_free, volatile int *dep_items, uint32_t tmem_base, volatile int *dead, int grp,
                                          int first, int step)
{
    constexpr int NBLK = S1 ? 8 : 16;
    constexpr int NQ = NBLK / 4;                     // slot groups per tile
    constexpr int WBYTES = kWBytes;
    static_assert(kProdWarps == 4, "one producer warp per slot of a group");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t stage0 = smem0 + kWBytes;
    const uint32_t ring0 = stage0 + kStages * kStageBytes;
    const int hj = grp >> 1, hl = grp & 1;           // S2 only: block group (16 blocks), output-row half
    const int n_tiles = p.tiles;
    if (first >= n_tiles) return;
    const uint32_t full0 = smem_u32(bar_full), empty0 = smem_u32(bar_empty);
    const uint32_t accf0 = smem_u32(bar_acc_full), acce0 = smem_u32(bar_acc_empty);

    if (warp >= kEpiWarps && warp < kEpiWarps + kProdWarps) {
        // ------------------------------------------------------------ producers: warp pw loads slot pw of every group
        const int pw = warp - kEpiWarps;
        if (lane != 0) return;
        if (pw == 0) {
            // resident weights of this CTA's group
            const uint32_t wbar = smem_u32(bar_w);
            mbar_expect_tx(wbar, WBYTES);
            if (S1) {
                for (int b = 0; b < 8; ++b) tma_load_2d(smem0 + b * 8192, &tm_R, 0, (grp * 8 + b) * kM, wbar);
            } else {
                for (int b = 0; b < 16; ++b)
                    tma_load_2d(smem0 + b * 4096, &tm_L, 0, (hj * 16 + b) * kM + hl * 32, wbar);
            }
        }
        RingBase<NQ> ring;
        int nitem_p = 0;
        [[maybe_unused]] int nitem_t = 0;
        for (int tile = first; tile < n_tiles; tile += step, ++nitem_t, ++nitem_p) {
            if (pw == 0) TRACE(0);
            if (!S1 && p.a > 0) {      // (a launch without stage-1 CTAs finds u' complete)
                if (pw == 0) {
                    // wait until all S1 groups have published their part of u' for this tile
                    const unsigned *ctr = p.counters + tile;
                    if (ld_acquire(ctr) < kS1Arrivals) {
                        const unsigned long long t0 = global_timer_ns();
                        while (ld_acquire(ctr) < kS1Arrivals) {
                            if (*dead || global_timer_ns() - t0 > kWaitLimitNs) {
                                *dead = 1;
                                atomicCAS(p.status, 0u, (unsigned)kErrPeerWait);
                                return;
                            }
                        }
                    }
                    // the last S2 group to get here clears the tile's counter for the next call
                    const unsigned old = atomicAdd(p.counters + tile, 1u);
                    if (old + 1 == kS1Arrivals + kS2Groups) atomicExch(p.counters + tile, 0u);
                    fence_proxy_async_global();
                    __threadfence_block();
                    *dep_items = nitem_p + 1;             // monotonic: cannot alias like a parity would
                } else {
                    if (*dep_items <= nitem_p) {
                        const unsigned long long t0 = global_timer_ns();
                        while (*dep_items <= nitem_p) {
                            if (*dead || global_timer_ns() - t0 > kWaitLimitNs) {
                                *dead = 1;
                                atomicCAS(p.status, 0u, (unsigned)kErrPeerWait);
                                return;
                            }
                        }
                    }
                    __threadfence_block();
                    fence_proxy_async_global();
                }
            }
            if (pw == 0) TRACE(1);
            const __nv_bfloat16 *usrc = p.u + ((long long)tile * 64 + hj * 16 + pw) * 4096;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                int g;
                uint32_t ph;
                ring.at(q, g, ph);
                if (!wait_fast(empty0 + g * 8, ph ^ 1, p.status, dead, kErrSlotWait)) return;
                const uint32_t full = full0 + g * 8;
                mbar_expect_tx(full, kSlotBytes);
                const uint32_t dst = ring0 + (g * 4 + pw) * kSlotBytes;
                if (S1) tma_load_2d(dst, &tm_x, (grp * 8 + q * 4 + pw) * kM, tile * 64, full);
                else bulk_load(dst, usrc + (size_t)q * 4 * 4096, 8192, full);
            }
            ring.next_tile();
            if (pw == 0) TRACE(2);
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------ MMA issuer (one thread issues every MMA)
        if (lane != 0) return;
        if (!mbar_wait(smem_u32(bar_w), 0, p.status, dead, kErrTmaWait)) return;
        tc_fence_after();
        RingBase<NQ> ring;
        uint32_t nitem = 0;
        [[maybe_unused]] int nitem_t = 0;
        // descriptor templates: only the 14-bit start-address field changes
        const uint64_t a_ring = (S1 ? make_smem_desc(0, 16, 1024, kSwizzle128) : make_smem_desc(0, 1024, 128, 0)) |
                                (uint64_t)(ring0 >> 4);
        const uint64_t b_res = make_smem_desc(0, 16, 1024, kSwizzle128) | (uint64_t)(smem0 >> 4);
        constexpr uint32_t idesc = make_idesc_bf16(64, S1 ? 64 : 32, 0, 0);
        constexpr int AK = S1 ? 2 : 128;             // K-step advance of the A descriptor (>>4 units)
        for (int tile = first; tile < n_tiles; tile += step, ++nitem_t, ++nitem) {
            // tiles alternate between two accumulator sets: lane halves (S1) or column halves (S2)
            const uint32_t buf = nitem & 1, par = (nitem >> 1) & 1;
            if (!wait_fast(acce0 + buf * 8, par ^ 1, p.status, dead, kErrTmemWait)) return;
            tc_fence_after();
            TRACE(3);
            const uint32_t dbase = S1 ? tmem_base + ((buf * 16) << 16) : tmem_base + buf * 256;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                int g;
                uint32_t ph;
                ring.at(q, g, ph);
                if (!wait_fast(full0 + g * 8, ph, p.status, dead, kErrTmaWait)) return;
                tc_fence_after();
                const uint64_t aq = a_ring + (uint64_t)(g * 4 * (kSlotBytes >> 4));
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int b = q * 4 + i;
                    const uint64_t ad = aq + i * (kSlotBytes >> 4);
                    const uint64_t bd = b_res + b * (S1 ? 512 : 256);
                    // S2: blocks 0-7 in lanes [0,16) of each sub-partition, 8-15 in lanes [16,32)
                    const uint32_t d = S1 ? dbase + b * 64 : dbase + ((uint32_t)((b >> 3) * 16) << 16) + (b & 7) * 32;
                    mma_f16_ss(d, ad, bd, idesc, 0);
                    mma_f16_ss(d, ad + AK, bd + 2, idesc, 1);
                    mma_f16_ss(d, ad + 2 * AK, bd + 4, idesc, 1);
                    mma_f16_ss(d, ad + 3 * AK, bd + 6, idesc, 1);
                }
                mma_commit(empty0 + g * 8);
            }
            mma_commit(accf0 + buf * 8);
            ring.next_tile();
            TRACE(4);
        }
    } else if (warp < kEpiWarps) {
        // ------------------------------------------------------------ epilogue (warps 0-7)
        // Two halves of four warps (one per TMEM sub-partition) take alternate chunks of a tile.  A chunk
        // is packed to bf16 into a staging buffer and handed to the half's store thread, which sends it
        // out with one TMA tensor store: global stores issued by these warps themselves would queue in
        // front of the tcgen05.mma issue (measured: they halve the MMA rate), bulk stores do not.
        const int q4 = warp & 3, sub = warp >> 2;      // TMEM sub-partition, epilogue half
        const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16);
        const int row = q4 * 16 + (lane & 15);         // token row of this thread within a tile
        const uint32_t my_stage = stage0 + sub * kStagesPerHalf * kStageBytes;
        const uint32_t stf0 = smem_u32(bar_st_full) + sub * kStagesPerHalf * 8;
        const uint32_t stfree0 = smem_u32(bar_st_free) + sub * kStagesPerHalf * 8;
        uint32_t nitem = 0, nchunk = 0;
        [[maybe_unused]] int nitem_t = 0;
        for (int tile = first; tile < n_tiles; tile += step, ++nitem_t, ++nitem) {
            const uint32_t buf = nitem & 1, par = (nitem >> 1) & 1;
            if (!wait_fast(accf0 + buf * 8, par, p.status, dead, kErrMmaWait)) return;
            tc_fence_after();
            if (threadIdx.x == 0) TRACE(5);
#pragma unroll 1
            for (int c = sub; c < 8; c += 2, ++nchunk) {
                const uint32_t k = nchunk & (kStagesPerHalf - 1);
                const uint32_t sbuf = my_stage + k * kStageBytes;
                // the store that last read this staging buffer must be done reading it
                if (!wait_fast(stfree0 + k * 8, ((nchunk / kStagesPerHalf) & 1) ^ 1, p.status, dead, kErrSlotWait))
                    return;
                if (S1) {
                    // accumulators of this tile live in lane half `buf`; chunk = 8 consecutive j
                    uint32_t v[8][8];
#pragma unroll
                    for (int kb = 0; kb < 8; ++kb) tmem_ld8(lane_base + kb * 64 + c * 8, v[kb]);
                    tmem_ld_wait();
                    if ((uint32_t)(lane >> 4) == buf) {
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const uint32_t o0 = pack_bf16(__uint_as_float(v[0][q]), __uint_as_float(v[1][q]));
                            const uint32_t o1 = pack_bf16(__uint_as_float(v[2][q]), __uint_as_float(v[3][q]));
                            const uint32_t o2 = pack_bf16(__uint_as_float(v[4][q]), __uint_as_float(v[5][q]));
                            const uint32_t o3 = pack_bf16(__uint_as_float(v[6][q]), __uint_as_float(v[7][q]));
                            // staging [j local 8][t 64][8 k]: the 1 KB slab of u'[tile][j][k/8 = g]
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sbuf + q * 1024 + row * 16),
                                         "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                        }
                    }
                } else {
                    // chunk = 4 consecutive output rows l; lanes i and i+16 hold blocks 0-7 and 8-15
                    uint32_t v[8][4];
#pragma unroll
                    for (int a = 0; a < 8; ++a) tmem_ld4(lane_base + buf * 256 + a * 32 + c * 4, v[a]);
                    tmem_ld_wait();
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint32_t o0 = pack_bf16(__uint_as_float(v[0][q]), __uint_as_float(v[1][q]));
                        const uint32_t o1 = pack_bf16(__uint_as_float(v[2][q]), __uint_as_float(v[3][q]));
                        const uint32_t o2 = pack_bf16(__uint_as_float(v[4][q]), __uint_as_float(v[5][q]));
                        const uint32_t o3 = pack_bf16(__uint_as_float(v[6][q]), __uint_as_float(v[7][q]));
                        // staging [l local 4][t 64][16 j]
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sbuf + q * 2048 + row * 32 + (lane >> 4) * 16),
                                     "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                    }
                }
                if (c + 2 >= 8) {
                    // last chunk of this half: the tile's accumulators have been read
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acce0 + buf * 8);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(stf0 + k * 8);
            }
            if (threadIdx.x == 0) { TRACE(6); TRACE(7); }
        }
    } else if (warp >= kStoreWarp0) {
        // ------------------------------------------------------------ store threads (one per epilogue half)
        const int sub = warp - kStoreWarp0;
        if (lane != 0) return;
        const uint32_t my_stage = stage0 + sub * kStagesPerHalf * kStageBytes;
        const uint32_t stf0 = smem_u32(bar_st_full) + sub * kStagesPerHalf * 8;
        const uint32_t stfree0 = smem_u32(bar_st_free) + sub * kStagesPerHalf * 8;
        uint32_t nchunk = 0;
        int pending = -1;                              // S1: tile whose stores still await publishing
        for (int tile = first; tile < n_tiles; tile += step) {
#pragma unroll 1
            for (int c = sub; c < 8; c += 2, ++nchunk) {
                const uint32_t k = nchunk & (kStagesPerHalf - 1);
                const uint32_t sbuf = my_stage + k * kStageBytes;
                if (!wait_fast(stf0 + k * 8, (nchunk / kStagesPerHalf) & 1, p.status, dead, kErrMmaWait)) return;
                if (S1) {
                    // u' as 8-byte words: [tile*64 + j][k/8][128 words]; 8 rows (j) of 1 KB
                    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(&tm_u),
                                 "r"(sbuf), "r"(0), "r"(grp), "r"(tile * 64 + c * 8) : "memory");
                } else {
                    // y as [l][t][j]: box 16 j x 64 t x 4 l; rows past the last token are clipped
                    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(&tm_y),
                                 "r"(sbuf), "r"(hj * 16), "r"(tile * 64), "r"(hl * 32 + c * 4) : "memory");
                }
                tma_store_commit();
                if (nchunk >= kStagesPerHalf - 1) {
                    // keep three stores in flight (a store's read latency is 1-2 thousand cycles); the
                    // buffer of the one before them is free again
                    tma_store_wait_read<kStagesPerHalf - 1>();
                    mbar_arrive(stfree0 + ((nchunk - (kStagesPerHalf - 1)) & (kStagesPerHalf - 1)) * 8);
                }
            }
            if (S1 && p.b > 0) {      // no stage-2 CTAs in the launch: nothing to publish to
                if (pending >= 0) {
                    // the previous tile's four stores are complete once at most four newer ones are pending
                    asm volatile("cp.async.bulk.wait_group 4;" ::: "memory");
                    fence_proxy_async_global();
                    __threadfence();
                    atomicAdd(p.counters + pending, 1u);
                }
                pending = tile;
            }
        }
        tma_store_wait_all<0>();
        if (S1 && p.b > 0 && pending >= 0) {
            fence_proxy_async_global();
            __threadfence();
            atomicAdd(p.counters + pending, 1u);
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
fused_fwd_m64_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_R,
                     const __grid_constant__ CUtensorMap tm_L, const __grid_constant__ CUtensorMap tm_u,
                     const __grid_constant__ CUtensorMap tm_y, const FwdParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kQuads], bar_empty[kQuads], bar_acc_full[2], bar_acc_empty[2], bar_w,
        bar_st_full[kStages], bar_st_free[kStages];
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead;
    __shared__ int dep_items;

    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5;

    // role of this CTA
    const int n_s1 = 8 * p.a;
    const bool is_s1 = (int)blockIdx.x < n_s1;
    const int grp = is_s1 ? (int)blockIdx.x % 8 : ((int)blockIdx.x - n_s1) % 8;
    const int first = is_s1 ? (int)blockIdx.x / 8 : ((int)blockIdx.x - n_s1) / 8;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kQuads; ++s) {
            mbar_init(smem_u32(&bar_full[s]), kProdWarps);   // four loads, one per producer warp
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        for (int h = 0; h < 2; ++h) {
            mbar_init(smem_u32(&bar_acc_full[h]), 1);
            mbar_init(smem_u32(&bar_acc_empty[h]), kEpiWarps);
        }
        mbar_init(smem_u32(&bar_w), 1);
        for (int k = 0; k < kStages; ++k) {
            mbar_init(smem_u32(&bar_st_full[k]), 4);    // the four warps of an epilogue half
            mbar_init(smem_u32(&bar_st_free[k]), 1);
        }
        fence_mbar_init();
        dead = 0;
        dep_items = 0;
        tma_prefetch_desc(is_s1 ? &tm_x : &tm_L);
        tma_prefetch_desc(is_s1 ? &tm_R : &tm_y);
        if (is_s1) tma_prefetch_desc(&tm_u);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    if (is_s1)
        role_body<true>(tm_x, tm_R, tm_L, tm_u, tm_y, p, smem0, bar_full, bar_empty, bar_acc_full, bar_acc_empty, &bar_w,
                        bar_st_full, bar_st_free, &dep_items, tmem_base, &dead, grp, first, p.a);
    else
        role_body<false>(tm_x, tm_R, tm_L, tm_u, tm_y, p, smem0, bar_full, bar_empty, bar_acc_full, bar_acc_empty, &bar_w,
                         bar_st_full, bar_st_free, &dep_items, tmem_base, &dead, grp, first, p.b);

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }

}  // namespace
}  // namespace tc

// Workspace: [status 256 B][tile counters, 64 KB][u' exchange buffer, tokens rounded up to 64].
constexpr size_t kFusedCounterBytes = 65536;

size_t fused_fwd_m64_workspace_bytes(int64_t tokens)
{
    // at least two tiles: the forward on clusters keeps its 1 MB of weight images where the exchange buffer starts
    const size_t tiles = tokens < 128 ? 2 : (size_t)((tokens + 63) / 64);
    return MONARCH_STATUS_BYTES + kFusedCounterBytes + tc::align256(tiles * 64 * (size_t)tc::kN * 2);
}

namespace {
// Launch with both stages (y != null) or with stage-1 CTAs only, which leaves P R x in `u` in the
// exchange layout [tile][j][k/8][t%64][k%8] for another kernel to consume.
int launch_fwd_m64(const void *x, const void *L, const void *R, void *y, void *u, unsigned *counters,
                   unsigned *status, int64_t tokens, cudaStream_t s)
{
    using namespace tc;
    const bool both = y != nullptr && x != nullptr;
    const bool s2_only = x == nullptr;
    const long long tiles = (tokens + 63) / 64;
    if (tiles * 4 > (long long)kFusedCounterBytes) return MONARCH_ERR_UNSUPPORTED;
    CUtensorMap tm_x, tm_R, tm_L, tm_u, tm_y;
    MONARCH_TRY(encode_tmap_2d(&tm_R, R, kN, kM, kM * 2, 64, 64, 128));
    if (s2_only) tm_x = tm_R;
    else MONARCH_TRY(encode_tmap_2d(&tm_x, x, (uint64_t)tokens, kN, kN * 2, 64, 64, 128));
    {
        // exchange buffer as 8-byte words [tile*64 + j][k/8][128]; a store moves 8 rows (j) of one k/8
        const uint64_t dims[3] = {128, 8, (uint64_t)tiles * 64}, strides[2] = {1024, 8192};
        const uint32_t box[3] = {128, 1, 8};
        MONARCH_TRY(encode_tmap_nd(&tm_u, u, 8, 3, dims, strides, box));
    }
    if (both || s2_only) {
        MONARCH_TRY(encode_tmap_2d(&tm_L, L, kN, kM, kM * 2, 32, 64, 128));
        // y as [l][t][j] bf16; a store moves 16 j x 64 t x 4 l
        const uint64_t ydims[3] = {64, (uint64_t)tokens, 64}, ystrides[2] = {(uint64_t)kN * 2, 128};
        const uint32_t ybox[3] = {16, 64, 4};
        MONARCH_TRY(encode_tmap_nd(&tm_y, y, 2, 3, ydims, ystrides, ybox));
    } else {
        tm_L = tm_R;
        tm_y = tm_u;
    }
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(fused_fwd_m64_kernel,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    FwdParams p;
    p.status = status;
    p.counters = counters;
    p.u = (__nv_bfloat16 *)u;
    p.y = (__nv_bfloat16 *)y;
    p.tokens = tokens;
    p.tiles = (int)tiles;
    // split the SMs between the stages: 8 R groups x a CTAs + 8 L groups x b CTAs.  Stage 2 issues
    // twice the MMAs (N = 32) and writes 32-byte pieces, so it gets about 60 % of the SMs.
    int a = both ? (sms * 2 + 20) / 40 : sms / 8;
    if (a < 1) a = 1;
    int b = both ? (sms - 8 * a) / 8 : 0;
    if (both && b < 1) b = 1;
    if (a > tiles) a = (int)tiles;
    if (b > tiles) b = (int)tiles;
    if (s2_only) { a = 0; b = sms / 8 < tiles ? sms / 8 : (int)tiles; if (b < 1) b = 1; }
    p.a = a;
    p.b = b;
    p.trace = nullptr;
#ifdef MONARCH_TRACE
    if (both == (getenv("MONARCH_TRACE_S1ONLY") == nullptr)) {
        if (const char *e = getenv("MONARCH_TRACE_PTR")) p.trace = (long long *)strtoull(e, nullptr, 0);
        if (both) {
            if (const char *e = getenv("MONARCH_SPLIT_A")) { p.a = atoi(e); p.b = (sms - 8 * p.a) / 8; }
            if (const char *e = getenv("MONARCH_SPLIT_B")) p.b = atoi(e);
        }
        if (p.a > tiles) p.a = (int)tiles;
        if (p.b > tiles) p.b = (int)tiles;
    }
#endif
    fused_fwd_m64_kernel<<<8 * p.a + 8 * p.b, kThreads, kSmemBytes, s>>>(tm_x, tm_R, tm_L, tm_u, tm_y, p);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}
}  // namespace

int fused_fwd_m64(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws,
                  cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
#ifdef MONARCH_TRACE
    // debug builds: comparison runs of the split schedule, as one launch or as one launch per stage
    static const bool two = getenv("MONARCH_TWO_LAUNCH") != nullptr;
    static const bool split = getenv("MONARCH_FWD_SPLIT") != nullptr;
    if (two) {
        void *u = (char *)ws + MONARCH_STATUS_BYTES + kFusedCounterBytes;
        MONARCH_TRY(launch_fwd_m64(x, nullptr, R, nullptr, u, nullptr, (unsigned *)ws, tokens, s));
        return launch_fwd_m64(nullptr, L, R, y, u, nullptr, (unsigned *)ws, tokens, s);
    }
    if (split)
        return launch_fwd_m64(x, L, R, y, (char *)ws + MONARCH_STATUS_BYTES + kFusedCounterBytes,
                              (unsigned *)((char *)ws + MONARCH_STATUS_BYTES), (unsigned *)ws, tokens, s);
#endif
    if (fused_fwd_m64_on_clusters()) {
        const int st = fused_fwd_m64_cluster(x, L, R, y, tokens, ws, s);
        if (st != MONARCH_ERR_UNSUPPORTED) return st;
    }
    return fused_fwd_m64_team(x, L, R, y, tokens, ws, s);
}

// The forward pass on clusters of four CTAs (the intermediate stays in distributed shared memory; nothing is left in
// the workspace for the backward call) when MONARCH_M64_CLUSTER is set.  Not the default: measured 80 us against
// 59 us (8192 tokens) and 273 against 180 us (32768 tokens) for the team schedule with its exchange through L2.
bool fused_fwd_m64_on_clusters()
{
    static const bool on = getenv("MONARCH_M64_CLUSTER") != nullptr;
    return on;
}

const void *fused_fwd_m64_saved_u(const void *fwd_ws)
{
    if (fused_fwd_m64_on_clusters()) return nullptr;
    return (const char *)fwd_ws + MONARCH_STATUS_BYTES + kFusedCounterBytes;
}

int fused_fwd_m64_stage1(const void *x, const void *R, void *u, int64_t tokens, unsigned *status,
                         cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    return launch_fwd_m64(x, nullptr, R, nullptr, u, nullptr, status, tokens, s);
}

}  // namespace monarch
