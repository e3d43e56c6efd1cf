// Fused backward kernels for m = 64 (n = 4096), bf16 in/out, fp32 accumulation in TMEM:
// dx = M^T dy = R^T P L^T P dy, and the all-in-one launch that also forms dL and dR.
//
// The mirror image of the fused forward kernel: persistent launches, CTAs (one per SM) specialise, 64-token
// tiles, tcgen05.mma with M = 64, the intermediate du handed over through an L2-resident exchange buffer that
// already has the operand layout of the consumer, outputs staged in shared memory and written by the TMA unit.
//
//   B1 CTAs (8 groups g of `b1` CTAs): du[t][k][j] = sum_l L[j][l][k] dy[t][l*64+j] for blocks j in [8g, 8g+8)
//       and all 64 columns k.  The outer permutation sits on the INPUT side here: block j needs column j of
//       every 64-element row segment.  TMA gathers the 16-byte pieces dy[t][l][8g..8g+8) as [64 t][16 l][8 j]
//       chunks; four warps turn each chunk into operand slices [j][l/8][t][l%8] with ldmatrix.trans / stmatrix
//       (an 8x8 16-bit transpose per instruction pair) - the only place in the library where the permutation
//       costs a pass over shared memory.  MMAs run in the transposed orientation D[k][t] (A = L_j^T from its
//       row-major tile, B = the slice), so that a thread of the epilogue finds the 8 blocks of its row side by
//       side and writes the 16 bytes du[t][k][8g..8g+8) of the exchange buffer [tile][k][j/8][t%64][j%8].
//   B2 CTAs (8 groups g of `b2` CTAs): dx[t][k*64+i] = sum_j R[k][j][i] du[t][k][j] for blocks
//       k in [8g, 8g+8).  One 8 KB bulk copy per block fetches du_k[64 x 64]; R_k is used transposed
//       from its row-major tile (MN-major, 128B swizzle); the result rows are 128 contiguous bytes per
//       (t, k), staged with the 128B swizzle and stored as 64 x 64 boxes.
//
// Waits are bounded; B1 waits on nothing outside its CTA, the other kinds on a per-tile counter bumped by B1.
#include <cstdio>
#include <cstdlib>

#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

constexpr int kM = 64;
constexpr int kN = kM * kM;
// warps: 0-7 epilogue, 8 control/loads, 9 MMA, 10-11 store threads, 12-15 transposers (B1) / loaders (B2),
// 16-17 write the transposed dy out when a caller wants it (B1)
constexpr int kEpiWarps = 8, kCtlWarp = 8, kMmaWarp = 9, kStoreWarp0 = 10, kAuxWarp0 = 12, kDypWarp = 16;
constexpr int kDypWarps = 2;
constexpr int kThreads = (kDypWarp + kDypWarps) * 32;
constexpr int kWBytes = 65536;                 // resident weights
constexpr int kStageBytes = 8192;
constexpr int kB2StagesPerHalf = 4;
constexpr int kRawBytes = 16384, kRawBufs = 4;                // B1: one K-step (16 l) of 8 blocks, as loaded
constexpr int kBlockSlice = 2048 + 16;                        // B1: one block's K-step operand, padded so that
constexpr int kSliceBytes = 8 * kBlockSlice;                  //     the 8 rows of an stmatrix hit 8 bank groups
constexpr int kOutRow = 1024 + 16;                            // B1: staged output row (64 tokens x 16 B), padded
constexpr int kOutBytes = 16 * kOutRow;                       //     one buffer per 16 rows k (TMEM quarter)
constexpr int kSlotBytes = 8192, kSlots = 12, kQuads = 3;     // B2 operand ring
constexpr int kSmemBytes = kWBytes + 65536 + 98304 + 1280 + 1024;  // 226.25 KB incl. alignment: B1 is the largest kind
static_assert(kWBytes + kRawBufs * kRawBytes + 2 * kSliceBytes + 4 * kOutBytes + 1024 <= kSmemBytes, "B1");
static_assert(kWBytes + 2 * kB2StagesPerHalf * kStageBytes + kSlots * kSlotBytes + 1024 <= kSmemBytes, "B2");
constexpr unsigned kB1Arrivals = 8 * 2;        // 8 B1 groups x 2 store warps per tile
constexpr unsigned kB2Groups = 8;

struct BwdParams {
    __nv_bfloat16 *du;         // exchange buffer [tiles][64 k][8][64 t][8] bf16
    __nv_bfloat16 *dyp;        // optional: P dy in the layout [tiles][64 j][8][64 t][8] (l = 8 * chunk + l%8)
    unsigned *counters;        // one per 64-token tile, zero between calls
    unsigned *status;
    long long tokens;
    int tiles;
    int b1, b2;                // CTAs per B1 group, per B2 group
    int b3;                    // all-in-one kernel: CTAs per group of the dL kind (0 elsewhere)
    int want_dx;               // all-in-one kernel: 0 = weight gradients only (dx is neither formed nor stored)
    unsigned need, reset_at;   // a tile is ready at `need` arrivals; the consumer that brings it to `reset_at` clears it
    const __nv_bfloat16 *dy;   // natural dy (for L2 prefetch hints only; the data path goes through TMA)
    const __nv_bfloat16 *u;    // all-in-one kernel: u' = P R x, [tiles][64 j][8][64 t][8] (forward exchange layout)
    float *dL, *dR;            // all-in-one kernel: gradients (added to)
    float *part_dL, *part_dR;  // all-in-one kernel, fixed summation order: every CTA stores its partial sums to slot
                               // [index within its group][64 blocks][64][64] instead of adding them to dL / dR (else null)
    long long *trace;          // optional per-CTA timeline (debug builds), else null
};

#ifdef MONARCH_TRACE
#define BTRACE(item, slot, val) do { if (p.trace && (item) < 16) p.trace[((size_t)blockIdx.x * 16 + (item)) * 8 + (slot)] = (val); } while (0)
#define BCLK() clock64()
#else
#define BTRACE(item, slot, val) do { } while (0)
#define BCLK() 0ll
#endif

struct Bars {
    uint64_t w;                               // resident weights landed
    uint64_t acc_full[2], acc_empty[2];       // TMEM accumulator sets
    uint64_t st_full[8], st_free[8];          // staging buffers (per half: B1 uses 2, B2 uses 4)
    uint64_t raw_full[4], raw_empty[4];       // B1 raw chunks
    uint64_t a_full[2], a_empty[2];           // B1 operand slices
    uint64_t full[4], empty[4];               // operand rings: groups of four slots (B2, dL kind) or pairs (B2R)
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
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *m, int x, int y, int z, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
        "l"(m), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ bool wait_fast(uint32_t bar, uint32_t parity, unsigned *status, volatile int *dead,
                                          unsigned code)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait(bar, parity, status, dead, code);
}
// bounded spin on a monotonic shared counter
__device__ __forceinline__ bool wait_count(volatile int *ctr, int need, unsigned *status, volatile int *dead)
{
    if (*ctr >= need) return true;
    const unsigned long long t0 = global_timer_ns();
    while (*ctr < need) {
        if (*dead || global_timer_ns() - t0 > kWaitLimitNs) {
            *dead = 1;
            atomicCAS(status, 0u, (unsigned)kErrPeerWait);
            return false;
        }
    }
    return true;
}

// Store thread shared by both kinds: sends staged chunks out with TMA tensor stores, keeps NST-1 of them
// in flight, and (B1) publishes a tile once its stores are complete.
template <bool B1, int NST, typename IssueFn>
__device__ __forceinline__ void store_thread(const BwdParams &p, Bars *bars, uint32_t stage0, int sub, int first,
                                             int step, volatile int *dead, IssueFn issue)
{
    const uint32_t my_stage = stage0 + sub * NST * kStageBytes;
    const uint32_t stf0 = smem_u32(bars->st_full) + sub * NST * 8;
    const uint32_t stfree0 = smem_u32(bars->st_free) + sub * NST * 8;
    uint32_t nchunk = 0;
    int pending = -1;
    for (int tile = first; tile < p.tiles; tile += step) {
#pragma unroll 1
        for (int c = sub; c < 8; c += 2, ++nchunk) {
            const uint32_t k = nchunk & (NST - 1);
            if (!wait_fast(stf0 + k * 8, (nchunk / NST) & 1, p.status, dead, kErrMmaWait)) return;
            issue(my_stage + k * kStageBytes, tile, c);
            tma_store_commit();
            if (nchunk >= NST - 1) {
                tma_store_wait_read<NST - 1>();
                mbar_arrive(stfree0 + ((nchunk - (NST - 1)) & (NST - 1)) * 8);
            }
        }
        if (B1 && p.b2 > 0) {     // no B2 CTAs in the launch: nothing to publish to
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
    if (B1 && p.b2 > 0 && pending >= 0) {
        fence_proxy_async_global();
        __threadfence();
        atomicAdd(p.counters + pending, 1u);
    }
}

// ------------------------------------------------------------------------------------------------ B1
// du^T_j = L_j^T (P dy)_j^T for the 8 blocks j of group g and all 64 columns k, in the "transposed" orientation
// D[k][t] (M = k, N = tokens): A = L_j^T straight from the resident row-major tile (MN-major, 128B swizzle),
// B = the transposed slice [l/8][t][l%8] (K-major, no swizzle).  A thread of the epilogue owns one row k and
// finds the 8 blocks j of its group side by side in TMEM, which is exactly the 16-byte piece
// du[t][k][8g..8g+8) of the exchange layout - no second group has to contribute to it.
__device__ __forceinline__ void b1_body(const CUtensorMap &tm_dy3, const CUtensorMap &tm_Lt, const BwdParams &p,
                                        uint32_t smem0, Bars *bars, uint32_t tmem_base, volatile int *dead, int grp,
                                        int first)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int step = p.b1;
    if (first >= p.tiles) return;
    const uint32_t raw0 = smem0 + kWBytes;
    const uint32_t a0 = raw0 + kRawBufs * kRawBytes;
    const uint32_t out0 = a0 + 2 * kSliceBytes;
    const uint32_t rawf = smem_u32(bars->raw_full), rawe = smem_u32(bars->raw_empty);
    const uint32_t af = smem_u32(bars->a_full), ae = smem_u32(bars->a_empty);
    const uint32_t accf0 = smem_u32(bars->acc_full), acce0 = smem_u32(bars->acc_empty);
    const uint32_t stf0 = smem_u32(bars->st_full), stfree0 = smem_u32(bars->st_free);

    if (warp == kCtlWarp) {
        if (lane != 0) return;
        // resident: the 8 blocks L_j of the group, row-major [l][k] with 128B swizzle
        const uint32_t wbar = smem_u32(&bars->w);
        mbar_expect_tx(wbar, kWBytes);
        for (int b = 0; b < 8; ++b) tma_load_2d(smem0 + b * 8192, &tm_Lt, 0, (grp * 8 + b) * kM, wbar);
        // gather: the 16-byte pieces dy[t][l][8g..8g+8) of one K-step (16 l) as [64 t][16 l][8 j]
        int rb = 0;
        uint32_t ph = 0;
        for (int tile = first; tile < p.tiles; tile += step) {
#pragma unroll 1
            for (int ks = 0; ks < 4; ++ks) {
                if (!wait_fast(rawe + rb * 8, ph ^ 1, p.status, dead, kErrSlotWait)) return;
                mbar_expect_tx(rawf + rb * 8, kRawBytes);
                tma_load_3d(raw0 + rb * kRawBytes, &tm_dy3, grp * 8, ks * 16, tile * 64, rawf + rb * 8);
                if (++rb == kRawBufs) { rb = 0; ph ^= 1; }
            }
        }
    } else if (warp >= kAuxWarp0 && warp < kAuxWarp0 + 4) {
        // transposers: raw [64 t][16 l][8 j]  ->  slices [8 j][2 l/8][64 t][8 l]; one ldmatrix.x4.trans /
        // stmatrix.x4 pair turns the 16 l x 8 j of two tokens
        const int tw = warp - kAuxWarp0;
        const int mi = lane >> 3, r = lane & 7;      // matrix of the x4 group, row within it
        const int lo = mi & 1, tt = mi >> 1;
        int rb = 0;
        uint32_t ph = 0, n = 0;
        [[maybe_unused]] long long w_raw = 0, w_ae = 0, w_tr = 0;
        for (int tile = first; tile < p.tiles; tile += step) {
#pragma unroll 1
            for (int ks = 0; ks < 4; ++ks, ++n) {
                const uint32_t ab = n & 1;
                [[maybe_unused]] const long long c0 = BCLK();
                if (!wait_fast(rawf + rb * 8, ph, p.status, dead, kErrTmaWait)) return;
                [[maybe_unused]] const long long c1 = BCLK();
                if (!wait_fast(ae + ab * 8, ((n >> 1) & 1) ^ 1, p.status, dead, kErrSlotWait)) return;
                [[maybe_unused]] const long long c2 = BCLK();
                w_raw += c1 - c0; w_ae += c2 - c1;
                const uint32_t src = raw0 + rb * kRawBytes + (tw * 16 + tt) * 256 + (lo * 8 + r) * 16;
                const uint32_t dst = a0 + ab * kSliceBytes + r * kBlockSlice + lo * 1024 + (tw * 16 + tt) * 16;
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    uint32_t m0, m1, m2, m3;
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(m0), "=r"(m1), "=r"(m2), "=r"(m3)
                                 : "r"(src + it * 512)
                                 : "memory");
                    asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(dst + it * 32),
                                 "r"(m0), "r"(m1), "r"(m2), "r"(m3)
                                 : "memory");
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(rawe + rb * 8);
                    mbar_arrive(af + ab * 8);
                }
                if (++rb == kRawBufs) { rb = 0; ph ^= 1; }
                w_tr += BCLK() - c2;
            }
            if (tw == 0 && lane == 0) {
                BTRACE((n >> 2) - 1, 1, w_raw); BTRACE((n >> 2) - 1, 2, w_ae); BTRACE((n >> 2) - 1, 3, w_tr);
            }
            w_raw = w_ae = w_tr = 0;
        }
    } else if (warp >= kDypWarp) {
        // the operand slices are P dy in 2 KB runs [l/8 2][t 64][8 l] per block j: copy them out with plain
        // coalesced stores (512 contiguous bytes per warp instruction; the TMA unit is busy gathering).  Each of
        // the copy warps takes half of the blocks; a slice buffer is free again when the MMAs and both have read it.
        const int dw = warp - kDypWarp;
        uint32_t n = 0;
        const bool want = p.dyp != nullptr;
        for (int tile = first; tile < p.tiles; tile += step) {
            char *dst = reinterpret_cast<char *>(p.dyp + ((long long)tile * 64 + grp * 8) * 4096) + lane * 16;
#pragma unroll 1
            for (int ks = 0; ks < 4; ++ks, ++n) {
                const uint32_t ab = n & 1;
                if (!wait_fast(af + ab * 8, (n >> 1) & 1, p.status, dead, kErrTmaWait)) return;
                if (want) {
                    const uint32_t src = a0 + ab * kSliceBytes + lane * 16;
#pragma unroll 4
                    for (int i = dw * 16; i < dw * 16 + 16; ++i) {
                        const int j = i >> 2, off = (i & 3) * 512;
                        uint4 v;
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                                     : "r"(src + j * kBlockSlice + off));
                        *reinterpret_cast<uint4 *>(dst + (long long)j * 8192 + ks * 2048 + off) = v;
                    }
                    __syncwarp();
                }
                if (lane == 0) mbar_arrive(ae + ab * 8);
            }
            if (want && p.b3 > 0) {
                // another kind of CTA of this launch reads P dy back: publish the tile
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(p.counters + tile, 1u);
            }
        }
    } else if (warp == kMmaWarp) {
        if (lane != 0) return;
        if (!mbar_wait(smem_u32(&bars->w), 0, p.status, dead, kErrTmaWait)) return;
        tc_fence_after();
        constexpr uint32_t idesc = make_idesc_bf16(64, 64, 1, 0);          // A = L_j^T: MN-major; B = slice: K-major
        const uint64_t a_mn = make_smem_desc(0, 16, 1024, kSwizzle128) | (uint64_t)(smem0 >> 4);
        const uint64_t b_ns = make_smem_desc(0, 1024, 128, 0);
        uint32_t n = 0, nitem = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            const uint32_t buf = nitem & 1, par = (nitem >> 1) & 1;
            [[maybe_unused]] const long long m0 = BCLK();
            if (!wait_fast(acce0 + buf * 8, par ^ 1, p.status, dead, kErrTmemWait)) return;
            tc_fence_after();
            [[maybe_unused]] long long w_af = 0;
            BTRACE(nitem, 0, BCLK() - m0);
            const uint32_t dbase = tmem_base + ((buf * 16) << 16);
#pragma unroll 1
            for (int ks = 0; ks < 4; ++ks, ++n) {
                const uint32_t ab = n & 1;
                [[maybe_unused]] const long long c0 = BCLK();
                if (!wait_fast(af + ab * 8, (n >> 1) & 1, p.status, dead, kErrTmaWait)) return;
                tc_fence_after();
                w_af += BCLK() - c0;
                const uint64_t as = a_mn + ks * 128;                          // 16 rows l of 128 B
                const uint64_t bs = b_ns | (uint64_t)((a0 + ab * kSliceBytes) >> 4);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    mma_f16_ss(dbase + j * 64, as + j * 512, bs + j * (kBlockSlice >> 4), idesc, ks != 0);
                mma_commit(ae + ab * 8);
            }
            mma_commit(accf0 + buf * 8);
            BTRACE(nitem, 4, w_af); BTRACE(nitem, 5, BCLK());
        }
    } else if (warp < kEpiWarps) {
        // lane -> row k = 16 q4 + lane % 16 of the tile in lane half `buf`; the two warps of a quarter take
        // 32 tokens each and fill one staging buffer [16 k][64 t][16 B] (rows padded against bank conflicts)
        const int q4 = warp & 3, sub = warp >> 2;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16);
        const uint32_t obuf = out0 + q4 * kOutBytes + (lane & 15) * kOutRow;
        uint32_t nitem = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            const uint32_t buf = nitem & 1, par = (nitem >> 1) & 1;
            if (!wait_fast(accf0 + buf * 8, par, p.status, dead, kErrMmaWait)) return;
            tc_fence_after();
            [[maybe_unused]] const long long e0 = BCLK();
            if (!wait_fast(stfree0 + q4 * 8, (nitem & 1) ^ 1, p.status, dead, kErrSlotWait)) return;
            if (threadIdx.x == 0) BTRACE(nitem, 6, BCLK() - e0);
            const bool mine = (uint32_t)(lane >> 4) == buf;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                const int t0 = sub * 32 + c * 8;
                uint32_t v[8][8];
#pragma unroll
                for (int b = 0; b < 8; ++b) tmem_ld8(lane_base + b * 64 + t0, v[b]);
                tmem_ld_wait();
                if (mine) {
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        const uint32_t o0 = pack_bf16(__uint_as_float(v[0][t]), __uint_as_float(v[1][t]));
                        const uint32_t o1 = pack_bf16(__uint_as_float(v[2][t]), __uint_as_float(v[3][t]));
                        const uint32_t o2 = pack_bf16(__uint_as_float(v[4][t]), __uint_as_float(v[5][t]));
                        const uint32_t o3 = pack_bf16(__uint_as_float(v[6][t]), __uint_as_float(v[7][t]));
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(obuf + (t0 + t) * 16),
                                     "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                    }
                }
            }
            tc_fence_before();
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(acce0 + buf * 8);
                mbar_arrive(stf0 + q4 * 8);
            }
            if (threadIdx.x == 0) BTRACE(nitem, 7, BCLK() - e0);
        }
    } else if (warp == kStoreWarp0 || warp == kStoreWarp0 + 1) {
        // copy the staged rows out: 1 KB per (k, group) into du[tile][k][j/8 = g][t][j%8].  Plain coalesced
        // stores (a warp writes 512 contiguous bytes), two quarters per warp: the TMA unit of a B1 SM is busy
        // gathering narrow rows, and bulk copies queued behind those gathers released the staging buffers
        // thousands of cycles late.
        const int sw = warp - kStoreWarp0;
        uint32_t nitem = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            char *dst = reinterpret_cast<char *>(p.du + (((long long)tile * 64) * 8 + grp) * 512);
#pragma unroll 1
            for (int qq = 0; qq < 2; ++qq) {
                const int q4 = sw * 2 + qq;
                if (!wait_fast(stf0 + q4 * 8, nitem & 1, p.status, dead, kErrMmaWait)) return;
#pragma unroll 4
                for (int i = 0; i < 32; ++i) {
                    const int r = i >> 1, off = (i & 1) * 512 + lane * 16;      // row k = 16 q4 + r, byte offset in it
                    uint4 v;
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                                 : "r"(out0 + q4 * kOutBytes + r * kOutRow + off));
                    *reinterpret_cast<uint4 *>(dst + (long long)(q4 * 16 + r) * 8192 + off) = v;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(stfree0 + q4 * 8);
            }
            if (p.b2 > 0) {
                // publish this warp's half of the tile (nothing to publish to in a launch without consumers)
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(p.counters + tile, 1u);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------ B2
__device__ __forceinline__ void b2_body(const CUtensorMap &tm_R, const CUtensorMap &tm_dx, const BwdParams &p,
                                        uint32_t smem0, Bars *bars, volatile int *dep_items, uint32_t tmem_base,
                                        volatile int *dead, int grp, int first)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int step = p.b2;
    if (first >= p.tiles) return;
    const uint32_t stage0 = smem0 + kWBytes;
    const uint32_t ring0 = stage0 + 2 * kB2StagesPerHalf * kStageBytes;
    const uint32_t full0 = smem_u32(bars->full), empty0 = smem_u32(bars->empty);
    const uint32_t accf0 = smem_u32(bars->acc_full), acce0 = smem_u32(bars->acc_empty);

    if (warp == kCtlWarp) {
        if (lane != 0) return;
        // resident: the 8 blocks R_k, row-major [j][i] with 128B swizzle
        const uint32_t wbar = smem_u32(&bars->w);
        mbar_expect_tx(wbar, kWBytes);
        for (int b = 0; b < 8; ++b) tma_load_2d(smem0 + b * 8192, &tm_R, 0, (grp * 8 + b) * kM, wbar);
        int nitem = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            // wait until all B1 groups have published their part of du for this tile
            const unsigned *ctr = p.counters + tile;
            if (ld_acquire(ctr) < p.need) {
                const unsigned long long t0 = global_timer_ns();
                while (ld_acquire(ctr) < p.need) {
                    if (*dead || global_timer_ns() - t0 > kWaitLimitNs) {
                        *dead = 1;
                        atomicCAS(p.status, 0u, (unsigned)kErrPeerWait);
                        return;
                    }
                }
            }
            // the last B2 group to get here clears the tile's counter for the next call
            const unsigned old = atomicAdd(p.counters + tile, 1u);
            if (old + 1 == p.reset_at) atomicExch(p.counters + tile, 0u);
            fence_proxy_async_global();
            __threadfence_block();
            *dep_items = nitem + 1;
        }
    } else if (warp >= kAuxWarp0 && warp < kAuxWarp0 + 4) {
        // loaders: warp pw fetches slot pw of every group of four
        if (lane != 0) return;
        const int pw = warp - kAuxWarp0;
        int quad = 0, nitem = 0;
        uint32_t phase = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            if (!wait_count(dep_items, nitem + 1, p.status, dead)) return;
            __threadfence_block();
            fence_proxy_async_global();
            const __nv_bfloat16 *src = p.du + ((long long)tile * 64 + grp * 8 + pw) * 4096;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                int g = quad + q;
                uint32_t ph = phase;
                if (g >= kQuads) { g -= kQuads; ph ^= 1; }
                if (!wait_fast(empty0 + g * 8, ph ^ 1, p.status, dead, kErrSlotWait)) return;
                mbar_expect_tx(full0 + g * 8, kSlotBytes);
                bulk_load(ring0 + (g * 4 + pw) * kSlotBytes, src + (size_t)q * 4 * 4096, 8192, full0 + g * 8);
            }
            quad += 2;
            if (quad >= kQuads) { quad -= kQuads; phase ^= 1; }
        }
    } else if (warp == kMmaWarp) {
        if (lane != 0) return;
        if (!mbar_wait(smem_u32(&bars->w), 0, p.status, dead, kErrTmaWait)) return;
        tc_fence_after();
        constexpr uint32_t idesc = make_idesc_bf16(64, 64, 0, 1);          // B = R_k^T: MN-major
        const uint64_t a_ring = make_smem_desc(0, 1024, 128, 0) | (uint64_t)(ring0 >> 4);
        const uint64_t b_mn = make_smem_desc(0, 16, 1024, kSwizzle128) | (uint64_t)(smem0 >> 4);
        int quad = 0;
        uint32_t phase = 0, nitem = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            const uint32_t buf = nitem & 1, par = (nitem >> 1) & 1;
            if (!wait_fast(acce0 + buf * 8, par ^ 1, p.status, dead, kErrTmemWait)) return;
            tc_fence_after();
            const uint32_t dbase = tmem_base + ((buf * 16) << 16);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                int g = quad + q;
                uint32_t ph = phase;
                if (g >= kQuads) { g -= kQuads; ph ^= 1; }
                if (!wait_fast(full0 + g * 8, ph, p.status, dead, kErrTmaWait)) return;
                tc_fence_after();
                const uint64_t aq = a_ring + (uint64_t)(g * 4 * (kSlotBytes >> 4));
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int b = q * 4 + i;
                    const uint64_t ad = aq + i * (kSlotBytes >> 4);
                    const uint64_t bd = b_mn + b * 512;
                    const uint32_t d = dbase + b * 64;
                    mma_f16_ss(d, ad, bd, idesc, 0);
                    mma_f16_ss(d, ad + 128, bd + 128, idesc, 1);             // 16 rows of 128 B per K-step
                    mma_f16_ss(d, ad + 256, bd + 256, idesc, 1);
                    mma_f16_ss(d, ad + 384, bd + 384, idesc, 1);
                }
                mma_commit(empty0 + g * 8);
            }
            mma_commit(accf0 + buf * 8);
            quad += 2;
            if (quad >= kQuads) { quad -= kQuads; phase ^= 1; }
        }
    } else if (warp < kEpiWarps) {
        const int q4 = warp & 3, sub = warp >> 2;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16);
        const int row = q4 * 16 + (lane & 15);
        constexpr int NST = kB2StagesPerHalf;
        const uint32_t my_stage = stage0 + sub * NST * kStageBytes;
        const uint32_t stf0 = smem_u32(bars->st_full) + sub * NST * 8;
        const uint32_t stfree0 = smem_u32(bars->st_free) + sub * NST * 8;
        uint32_t nitem = 0, nchunk = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            const uint32_t buf = nitem & 1, par = (nitem >> 1) & 1;
            if (!wait_fast(accf0 + buf * 8, par, p.status, dead, kErrMmaWait)) return;
            tc_fence_after();
            const bool mine = (uint32_t)(lane >> 4) == buf;
#pragma unroll 1
            for (int c = sub; c < 8; c += 2, ++nchunk) {
                const uint32_t k = nchunk & (NST - 1);
                const uint32_t sbuf = my_stage + k * kStageBytes;
                if (!wait_fast(stfree0 + k * 8, ((nchunk / NST) & 1) ^ 1, p.status, dead, kErrSlotWait)) return;
                // chunk = block c: 64 contiguous outputs dx[t][(8g+c)*64 ..] per token
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t v[2][16];
                    tmem_ld16(lane_base + c * 64 + h * 32, v[0]);
                    tmem_ld16(lane_base + c * 64 + h * 32 + 16, v[1]);
                    tmem_ld_wait();
                    if (mine) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint32_t *w = &v[e >> 1][(e & 1) * 8];
                            const uint32_t o0 = pack_bf16(__uint_as_float(w[0]), __uint_as_float(w[1]));
                            const uint32_t o1 = pack_bf16(__uint_as_float(w[2]), __uint_as_float(w[3]));
                            const uint32_t o2 = pack_bf16(__uint_as_float(w[4]), __uint_as_float(w[5]));
                            const uint32_t o3 = pack_bf16(__uint_as_float(w[6]), __uint_as_float(w[7]));
                            const int ch = h * 4 + e;                          // 16-byte chunk of the 128-byte row
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sbuf + row * 128 + ((ch ^ (row & 7)) * 16)),
                                         "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                        }
                    }
                }
                if (c + 2 >= 8) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acce0 + buf * 8);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(stf0 + k * 8);
            }
        }
    } else if (warp >= kStoreWarp0 && warp < kStoreWarp0 + 2) {
        if (lane != 0) return;
        const int sub = warp - kStoreWarp0;
        store_thread<false, kB2StagesPerHalf>(p, bars, stage0, sub, first, step, dead,
            [&](uint32_t sbuf, int tile, int c) { tma_store_2d(&tm_dx, sbuf, (grp * 8 + c) * kM, tile * 64); });
    }
}

__global__ void __launch_bounds__(kThreads, 1)
fused_bwd_dx_m64_kernel(const __grid_constant__ CUtensorMap tm_dy3, const __grid_constant__ CUtensorMap tm_Lt,
                        const __grid_constant__ CUtensorMap tm_R, const __grid_constant__ CUtensorMap tm_du,
                        const __grid_constant__ CUtensorMap tm_dx, const BwdParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) Bars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead;
    __shared__ int dep_items;

    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5;
    const int n_b1 = 8 * p.b1;
    const bool is_b1 = (int)blockIdx.x < n_b1;
    const int grp = is_b1 ? (int)blockIdx.x % 8 : ((int)blockIdx.x - n_b1) % 8;
    const int first = is_b1 ? (int)blockIdx.x / 8 : ((int)blockIdx.x - n_b1) / 8;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars.w), 1);
        for (int h = 0; h < 2; ++h) {
            mbar_init(smem_u32(&bars.acc_full[h]), 1);
            mbar_init(smem_u32(&bars.acc_empty[h]), kEpiWarps);
            mbar_init(smem_u32(&bars.a_full[h]), 4);
            mbar_init(smem_u32(&bars.a_empty[h]), 1 + kDypWarps);   // MMA commit + the copy-out warps
        }
        for (int h = 0; h < 4; ++h) {
            mbar_init(smem_u32(&bars.raw_full[h]), 1);
            mbar_init(smem_u32(&bars.raw_empty[h]), 4);      // the four transposer warps
        }
        for (int k = 0; k < 8; ++k) {
            // B1: the two warps of a TMEM quarter; B2: the four warps of an epilogue half
            mbar_init(smem_u32(&bars.st_full[k]), is_b1 ? 2 : 4);
            mbar_init(smem_u32(&bars.st_free[k]), 1);
        }
        for (int q = 0; q < 4; ++q) {
            mbar_init(smem_u32(&bars.full[q]), 4);           // four loads, one per loader warp
            mbar_init(smem_u32(&bars.empty[q]), 1);
        }
        fence_mbar_init();
        dead = 0;
        dep_items = 0;
        if (is_b1) { tma_prefetch_desc(&tm_dy3); tma_prefetch_desc(&tm_Lt); }
        else { tma_prefetch_desc(&tm_R); tma_prefetch_desc(&tm_dx); }
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    if (is_b1) b1_body(tm_dy3, tm_Lt, p, smem0, &bars, tmem_base, &dead, grp, first);
    else b2_body(tm_R, tm_dx, p, smem0, &bars, &dep_items, tmem_base, &dead, grp, first);

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}


// ------------------------------------------------------------------------------------------------ all-in-one kernel
// dx, dL and dR in one launch: B1 CTAs as above (writing du and P dy to their L2-resident exchange buffers),
// "B2R" CTAs that turn the du slabs of 8 blocks k into dx AND into dR (the same 8 KB of shared memory is the
// K-major A operand of dx = du R and, read token-major, the A operand of dR += du^T x), and "WL" CTAs that
// reduce dL += (P dy)^T u' for 16 blocks j.  Every consumer waits on the tile's counter, so du and P dy are read
// back from L2 a few thousand cycles after they were written.

__device__ __forceinline__ bool wait_tile(const BwdParams &p, int tile, volatile int *dead)
{
    const unsigned *ctr = p.counters + tile;
    if (ld_acquire(ctr) < p.need) {
        const unsigned long long t0 = global_timer_ns();
        while (ld_acquire(ctr) < p.need) {
            if (*dead || global_timer_ns() - t0 > kWaitLimitNs) {
                *dead = 1;
                atomicCAS(p.status, 0u, (unsigned)kErrPeerWait);
                return false;
            }
        }
    }
    const unsigned old = atomicAdd(p.counters + tile, 1u);
    if (old + 1 == p.reset_at) atomicExch(p.counters + tile, 0u);
    fence_proxy_async_global();
    __threadfence_block();
    return true;
}

// A weight gradient's sums leave TMEM through shared memory and tiled TMA copies (boxes of 16 rows x 32 fp32 columns,
// 128-byte rows, swizzled): added to the gradient in L2, or stored to this CTA's slot of the partial sums.  Plain
// 16-byte reductions from the epilogue threads, each to its own 256-byte row, took 8 us of the call.
__device__ __forceinline__ void grad_box_out(const CUtensorMap *m, uint32_t src, int x, int y, bool store)
{
    if (store)
        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(m), "r"(src), "r"(x), "r"(y)
                     : "memory");
    else
        asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(m),
                     "r"(src), "r"(x), "r"(y)
                     : "memory");
}
// One warp, one block iteration: lanes with `active` hold 32 columns (v) of row r16 (0..15) of their block; `box` is
// this lane's 2 KB box in the warp's staging area.
__device__ __forceinline__ void grad_stage_row(uint32_t box, int r16, const uint32_t (&v)[2][16])
{
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const uint32_t *w = &v[e >> 2][(e & 3) * 4];
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(box + r16 * 128 + ((e ^ (r16 & 7)) << 4)), "r"(w[0]), "r"(w[1]),
                     "r"(w[2]), "r"(w[3]) : "memory");
    }
}

constexpr int kRSlotBytes = 16384;               // B2R / WL ring slot: two 8 KB operands of one block

__device__ __forceinline__ void b2r_body(const CUtensorMap &tm_R, const CUtensorMap &tm_x, const CUtensorMap &tm_dx,
                                         const CUtensorMap &tm_gR, const BwdParams &p, uint32_t smem0, Bars *bars, volatile int *dep_items,
                                         uint32_t tmem_base, volatile int *dead, int grp, int first)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int step = p.b2;
    if (first >= p.tiles) return;
    constexpr int NST = 2;                                             // staging buffers per epilogue half
    const uint32_t stage0 = smem0 + kWBytes;
    const uint32_t ring0 = stage0 + 2 * NST * kStageBytes;              // 8 slots x 16 KB, handed over in pairs
    const uint32_t full0 = smem_u32(bars->full), empty0 = smem_u32(bars->empty);
    const uint32_t dxf = smem_u32(&bars->acc_full[0]), dxe = smem_u32(&bars->acc_empty[0]);
    const uint32_t drf = smem_u32(&bars->acc_full[1]);

    if (warp == kCtlWarp) {
        if (lane != 0) return;
        const uint32_t wbar = smem_u32(&bars->w);
        mbar_expect_tx(wbar, kWBytes);
        for (int b = 0; b < 8; ++b) tma_load_2d(smem0 + b * 8192, &tm_R, 0, (grp * 8 + b) * kM, wbar);
        int nitem = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            if (!wait_tile(p, tile, dead)) return;
            *dep_items = nitem + 1;
        }
    } else if (warp >= kAuxWarp0 && warp < kAuxWarp0 + 2) {
        // loaders: warp pw fills slot pw of every pair with (du slab, x tile) of block 2g + pw
        if (lane != 0) return;
        const int pw = warp - kAuxWarp0;
        int nitem = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            if (!wait_count(dep_items, nitem + 1, p.status, dead)) return;
            __threadfence_block();
            fence_proxy_async_global();
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const int b = g * 2 + pw;
                if (!wait_fast(empty0 + g * 8, (nitem & 1) ^ 1, p.status, dead, kErrSlotWait)) return;
                mbar_expect_tx(full0 + g * 8, kRSlotBytes);
                const uint32_t slot = ring0 + b * kRSlotBytes;
                bulk_load(slot, p.du + ((long long)tile * 64 + grp * 8 + b) * 4096, 8192, full0 + g * 8);
                tma_load_2d(slot + 8192, &tm_x, (grp * 8 + b) * kM, tile * 64, full0 + g * 8);
            }
        }
    } else if (warp == kMmaWarp) {
        if (lane != 0) return;
        if (!mbar_wait(smem_u32(&bars->w), 0, p.status, dead, kErrTmaWait)) return;
        tc_fence_after();
        constexpr uint32_t idesc_dx = make_idesc_bf16(64, 64, 0, 1);       // A = du (K = j), B = R_k^T
        constexpr uint32_t idesc_dr = make_idesc_bf16(64, 64, 1, 1);       // A = du^T (K = t), B = x (K = t)
        const uint64_t a_dx = make_smem_desc(0, 1024, 128, 0) | (uint64_t)(ring0 >> 4);
        const uint64_t b_dx = make_smem_desc(0, 16, 1024, kSwizzle128) | (uint64_t)(smem0 >> 4);
        const uint64_t a_dr = make_smem_desc(0, 128, 1024, 0) | (uint64_t)(ring0 >> 4);
        const uint64_t b_dr = make_smem_desc(0, 16, 1024, kSwizzle128) | (uint64_t)((ring0 + 8192) >> 4);
        uint32_t nitem = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            if (p.want_dx) {
                // dx of this tile: the single accumulator set must have been drained
                if (!wait_fast(dxe, (nitem & 1) ^ 1, p.status, dead, kErrTmemWait)) return;
                tc_fence_after();
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    if (!wait_fast(full0 + g * 8, nitem & 1, p.status, dead, kErrTmaWait)) return;
                    tc_fence_after();
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int b = g * 2 + i;
                        const uint64_t ad = a_dx + (uint64_t)(b * (kRSlotBytes >> 4));
                        const uint64_t bd = b_dx + b * 512;
                        const uint32_t d = tmem_base + b * 64;
                        mma_f16_ss(d, ad, bd, idesc_dx, 0);
                        mma_f16_ss(d, ad + 128, bd + 128, idesc_dx, 1);
                        mma_f16_ss(d, ad + 256, bd + 256, idesc_dx, 1);
                        mma_f16_ss(d, ad + 384, bd + 384, idesc_dx, 1);
                    }
                }
                mma_commit(dxf);
            }
            // dR += du^T x while the epilogue drains dx; each pair of slots is released after its last use
            const uint32_t acc = nitem != 0;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                if (!p.want_dx) {      // (with dx the operands of the pair were awaited above)
                    if (!wait_fast(full0 + g * 8, nitem & 1, p.status, dead, kErrTmaWait)) return;
                    tc_fence_after();
                }
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int b = g * 2 + i;
                    const uint64_t ad = a_dr + (uint64_t)(b * (kRSlotBytes >> 4));
                    const uint64_t bd = b_dr + (uint64_t)(b * (kRSlotBytes >> 4));
                    const uint32_t d = tmem_base + ((uint32_t)16 << 16) + b * 64;
                    mma_f16_ss(d, ad, bd, idesc_dr, acc);
                    mma_f16_ss(d, ad + 16, bd + 128, idesc_dr, 1);
                    mma_f16_ss(d, ad + 32, bd + 256, idesc_dr, 1);
                    mma_f16_ss(d, ad + 48, bd + 384, idesc_dr, 1);
                }
                mma_commit(empty0 + g * 8);
            }
        }
        mma_commit(drf);
    } else if (warp < kEpiWarps) {
        const int q4 = warp & 3, sub = warp >> 2;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16);
        const int row = q4 * 16 + (lane & 15);
        const uint32_t my_stage = stage0 + sub * NST * kStageBytes;
        const uint32_t stf0 = smem_u32(bars->st_full) + sub * NST * 8;
        const uint32_t stfree0 = smem_u32(bars->st_free) + sub * NST * 8;
        const bool mine = lane < 16;                                       // dx lives in the first 16 lanes of each quarter
        uint32_t nitem = 0, nchunk = 0;
        for (int tile = first; p.want_dx && tile < p.tiles; tile += step, ++nitem) {
            if (!wait_fast(dxf, nitem & 1, p.status, dead, kErrMmaWait)) return;
            tc_fence_after();
#pragma unroll 1
            for (int c = sub; c < 8; c += 2, ++nchunk) {
                const uint32_t k = nchunk & (NST - 1);
                const uint32_t sbuf = my_stage + k * kStageBytes;
                if (!wait_fast(stfree0 + k * 8, ((nchunk / NST) & 1) ^ 1, p.status, dead, kErrSlotWait)) return;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint32_t v[2][16];
                    tmem_ld16(lane_base + c * 64 + h * 32, v[0]);
                    tmem_ld16(lane_base + c * 64 + h * 32 + 16, v[1]);
                    tmem_ld_wait();
                    if (mine) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint32_t *w = &v[e >> 1][(e & 1) * 8];
                            const uint32_t o0 = pack_bf16(__uint_as_float(w[0]), __uint_as_float(w[1]));
                            const uint32_t o1 = pack_bf16(__uint_as_float(w[2]), __uint_as_float(w[3]));
                            const uint32_t o2 = pack_bf16(__uint_as_float(w[4]), __uint_as_float(w[5]));
                            const uint32_t o3 = pack_bf16(__uint_as_float(w[6]), __uint_as_float(w[7]));
                            const int ch = h * 4 + e;
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sbuf + row * 128 + ((ch ^ (row & 7)) * 16)),
                                         "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                        }
                    }
                }
                if (c + 2 >= 8) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(dxe);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(stf0 + k * 8);
            }
        }
        // dR partial sums of this CTA's tiles: lanes 16-31 of each quarter hold row 16 q4 + lane - 16 of block b.  The
        // operand ring is idle by now: every warp stages its 16 rows of a block there (two boxes of 32 columns, two
        // buffers in turn) and its lane 0 sends them off
        if (!mbar_wait(drf, 0, p.status, dead, kErrMmaWait)) return;
        tc_fence_after();
        const bool part = p.part_dR != nullptr;
        const uint32_t wst = ring0 + warp * 8192;
        const int row0 = (part ? first * 4096 : 0) + (grp * 8) * 64 + q4 * 16;
        int it = 0;
#pragma unroll 1
        for (int b = sub * 4; b < sub * 4 + 4; ++b, ++it) {
            const uint32_t buf = wst + (it & 1) * 4096;
            if (it >= 2) {
                if (lane == 0) tma_store_wait_read<1>();
                __syncwarp();
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t v[2][16];
                tmem_ld16(lane_base + b * 64 + h * 32, v[0]);
                tmem_ld16(lane_base + b * 64 + h * 32 + 16, v[1]);
                tmem_ld_wait();
                if (!mine) grad_stage_row(buf + h * 2048, lane & 15, v);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                grad_box_out(&tm_gR, buf, 0, row0 + b * 64, part);
                grad_box_out(&tm_gR, buf + 2048, 32, row0 + b * 64, part);
                tma_store_commit();
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
    } else if (warp >= kStoreWarp0 && warp < kStoreWarp0 + 2) {
        if (lane != 0 || !p.want_dx) return;
        const int sub = warp - kStoreWarp0;
        store_thread<false, NST>(p, bars, stage0, sub, first, step, dead,
            [&](uint32_t sbuf, int tile, int c) { tma_store_2d(&tm_dx, sbuf, (grp * 8 + c) * kM, tile * 64); });
    }
}

__device__ __forceinline__ void wl_body(const CUtensorMap &tm_gL, const BwdParams &p, uint32_t ring0, Bars *bars, volatile int *dep_items,
                                        uint32_t tmem_base, volatile int *dead, int grp, int first)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int step = p.b3, blk0 = grp * 16;
    if (first >= p.tiles) return;
    const uint32_t full0 = smem_u32(bars->full), empty0 = smem_u32(bars->empty);
    const uint32_t accf = smem_u32(&bars->acc_full[0]);

    if (warp == kCtlWarp) {
        if (lane != 0) return;
        int nitem = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            if (!wait_tile(p, tile, dead)) return;
            *dep_items = nitem + 1;
        }
    } else if (warp >= kAuxWarp0 && warp < kAuxWarp0 + 4) {
        // loader pw fetches slot pw of every group of four: (P dy slab, u' slab) of block blk0 + 4q + pw
        if (lane != 0) return;
        const int pw = warp - kAuxWarp0;
        int g = 0, nitem = 0;
        uint32_t ph = 0;
        for (int tile = first; tile < p.tiles; tile += step, ++nitem) {
            if (!wait_count(dep_items, nitem + 1, p.status, dead)) return;
            __threadfence_block();
            fence_proxy_async_global();
#pragma unroll 1
            for (int q = 0; q < 4; ++q) {
                if (!wait_fast(empty0 + g * 8, ph ^ 1, p.status, dead, kErrSlotWait)) return;
                const uint32_t slot = ring0 + (g * 4 + pw) * kRSlotBytes;
                const long long run = ((long long)tile * 64 + blk0 + q * 4 + pw) * 4096;
                mbar_expect_tx(full0 + g * 8, kRSlotBytes);
                bulk_load(slot, p.dyp + run, 8192, full0 + g * 8);
                bulk_load(slot + 8192, p.u + run, 8192, full0 + g * 8);
                if (++g == kQuads) { g = 0; ph ^= 1; }
            }
        }
    } else if (warp == kMmaWarp) {
        if (lane != 0) return;
        constexpr uint32_t idesc = make_idesc_bf16(64, 64, 1, 1);          // both operands token-major
        const uint64_t d_run = make_smem_desc(0, 128, 1024, 0);
        const uint64_t a_base = d_run | (uint64_t)(ring0 >> 4);
        const uint64_t b_base = d_run | (uint64_t)((ring0 + 8192) >> 4);
        int g = 0;
        uint32_t ph = 0;
        for (int tile = first; tile < p.tiles; tile += step) {
            const uint32_t acc = tile != first;
#pragma unroll 1
            for (int q = 0; q < 4; ++q) {
                if (!wait_fast(full0 + g * 8, ph, p.status, dead, kErrTmaWait)) return;
                tc_fence_after();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int b = q * 4 + i;
                    const uint32_t d = tmem_base + ((uint32_t)((b >> 3) * 16) << 16) + (b & 7) * 64;
                    const uint64_t ad = a_base + (uint64_t)((g * 4 + i) * (kRSlotBytes >> 4));
                    const uint64_t bd = b_base + (uint64_t)((g * 4 + i) * (kRSlotBytes >> 4));
                    mma_f16_ss(d, ad, bd, idesc, acc);
                    mma_f16_ss(d, ad + 16, bd + 16, idesc, 1);
                    mma_f16_ss(d, ad + 32, bd + 32, idesc, 1);
                    mma_f16_ss(d, ad + 48, bd + 48, idesc, 1);
                }
                mma_commit(empty0 + g * 8);
                if (++g == kQuads) { g = 0; ph ^= 1; }
            }
        }
        mma_commit(accf);
    } else if (warp < kEpiWarps) {
        const int q4 = warp & 3, sub = warp >> 2;
        if (!mbar_wait(accf, 0, p.status, dead, kErrMmaWait)) return;
        tc_fence_after();
        const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16);
        // lanes 0-15 hold rows 16 q4 + lane of block blk0 + b, lanes 16-31 the same rows of block blk0 + 8 + b; staging
        // in the idle operand ring as in the dR flush: four boxes (two blocks x two halves of the columns) per step
        const bool part = p.part_dL != nullptr;
        const uint32_t wst = ring0 + warp * 16384;
        const int sel = lane >> 4;
        const int row0 = (part ? first * 4096 : 0) + blk0 * 64 + q4 * 16;
        int it = 0;
#pragma unroll 1
        for (int b = sub * 4; b < sub * 4 + 4; ++b, ++it) {
            const uint32_t buf = wst + (it & 1) * 8192;
            if (it >= 2) {
                if (lane == 0) tma_store_wait_read<1>();
                __syncwarp();
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t v[2][16];
                tmem_ld16(lane_base + b * 64 + h * 32, v[0]);
                tmem_ld16(lane_base + b * 64 + h * 32 + 16, v[1]);
                tmem_ld_wait();
                grad_stage_row(buf + (sel * 2 + h) * 2048, lane & 15, v);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    grad_box_out(&tm_gL, buf + k * 2048, (k & 1) * 32, row0 + ((k >> 1) * 8 + b) * 64, part);
                tma_store_commit();
            }
        }
        if (lane == 0) tma_store_wait_all<0>();
    }
}

__global__ void __launch_bounds__(kThreads, 1)
fused_bwd_all_m64_kernel(const __grid_constant__ CUtensorMap tm_dy3, const __grid_constant__ CUtensorMap tm_Lt,
                         const __grid_constant__ CUtensorMap tm_R, const __grid_constant__ CUtensorMap tm_du,
                         const __grid_constant__ CUtensorMap tm_dx, const __grid_constant__ CUtensorMap tm_x,
                         const __grid_constant__ CUtensorMap tm_gL, const __grid_constant__ CUtensorMap tm_gR,
                         const BwdParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) Bars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead;
    __shared__ int dep_items;

    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5;
    const int n_b1 = 8 * p.b1, n_b2 = 8 * p.b2;
    const int bid = (int)blockIdx.x;
    const int kind = bid < n_b1 ? 0 : bid < n_b1 + n_b2 ? 1 : 2;
    const int idx = kind == 0 ? bid : kind == 1 ? bid - n_b1 : bid - n_b1 - n_b2;
    const int grp = kind == 2 ? idx % 4 : idx % 8;
    const int first = kind == 2 ? idx / 4 : idx / 8;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars.w), 1);
        for (int h = 0; h < 2; ++h) {
            mbar_init(smem_u32(&bars.acc_full[h]), 1);
            mbar_init(smem_u32(&bars.acc_empty[h]), kEpiWarps);
            mbar_init(smem_u32(&bars.a_full[h]), 4);
            mbar_init(smem_u32(&bars.a_empty[h]), 1 + kDypWarps);   // MMA commit + the copy-out warps
        }
        for (int h = 0; h < 4; ++h) {
            mbar_init(smem_u32(&bars.raw_full[h]), 1);
            mbar_init(smem_u32(&bars.raw_empty[h]), 4);
        }
        for (int k = 0; k < 8; ++k) {
            mbar_init(smem_u32(&bars.st_full[k]), kind == 0 ? 2 : 4);
            mbar_init(smem_u32(&bars.st_free[k]), 1);
        }
        for (int q = 0; q < 4; ++q) {
            mbar_init(smem_u32(&bars.full[q]), kind == 1 ? 2 : 4);   // loads per group: a pair (B2R) or four (WL)
            mbar_init(smem_u32(&bars.empty[q]), 1);
        }
        fence_mbar_init();
        dead = 0;
        dep_items = 0;
        if (kind == 0) { tma_prefetch_desc(&tm_dy3); tma_prefetch_desc(&tm_Lt); }
        else if (kind == 1) { tma_prefetch_desc(&tm_R); tma_prefetch_desc(&tm_dx); tma_prefetch_desc(&tm_x); tma_prefetch_desc(&tm_gR); }
        else tma_prefetch_desc(&tm_gL);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    if (kind == 0) b1_body(tm_dy3, tm_Lt, p, smem0, &bars, tmem_base, &dead, grp, first);
    else if (kind == 1) b2r_body(tm_R, tm_x, tm_dx, tm_gR, p, smem0, &bars, &dep_items, tmem_base, &dead, grp, first);
    else wl_body(tm_gL, p, smem0, &bars, &dep_items, tmem_base, &dead, grp, first);

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

}  // namespace
}  // namespace tc

constexpr size_t kBwdCounterBytes = 65536;

size_t fused_bwd_dx_m64_workspace_bytes(int64_t tokens)
{
    const size_t tiles = (size_t)((tokens + 63) / 64);
    return MONARCH_STATUS_BYTES + kBwdCounterBytes + ((tiles * 64 * (size_t)tc::kN * 2 + 255) & ~(size_t)255);
}

namespace {
// Launch with both stages (dx != null) or with B1 CTAs only, which leaves du in the exchange layout
// [tile][k][j/8][t%64][j%8] (and, if `dyp` is given, P dy as [tile][j][l/8][t%64][l%8]) for another
// kernel to consume.
int launch_bwd_m64(const void *dy, const void *L, const void *R, void *dx, void *du, void *dyp,
                   unsigned *counters, unsigned *status, int64_t tokens, cudaStream_t s)
{
    using namespace tc;
    const bool both = dx != nullptr;
    const long long tiles = (tokens + 63) / 64;
    if (tiles * 4 > (long long)kBwdCounterBytes) return MONARCH_ERR_UNSUPPORTED;
    CUtensorMap tm_dy3, tm_Lt, tm_R, tm_du, tm_dx;
    {
        // dy as [t][l][j]: a load brings 8 j x 16 l x 64 t (16-byte pieces)
        const uint64_t dims[3] = {64, 64, (uint64_t)tokens}, strides[2] = {128, (uint64_t)kN * 2};
        const uint32_t box[3] = {8, 16, 64};
        MONARCH_TRY(encode_tmap_nd(&tm_dy3, dy, 2, 3, dims, strides, box));
        // exchange buffer as 8-byte words [tile*64 + k][j/8][128]; a store moves 4 k x 2 j/8 x 1 KB
        const uint64_t udims[3] = {128, 8, (uint64_t)tiles * 64}, ustrides[2] = {1024, 8192};
        const uint32_t ubox[3] = {128, 2, 4};
        MONARCH_TRY(encode_tmap_nd(&tm_du, du, 8, 3, udims, ustrides, ubox));
    }
    MONARCH_TRY(encode_tmap_2d(&tm_Lt, L, kN, kM, kM * 2, 64, 64, 128));     // [64 l][64 k] per block, 128B swizzle
    if (both) {
        MONARCH_TRY(encode_tmap_2d(&tm_R, R, kN, kM, kM * 2, 64, 64, 128));
        MONARCH_TRY(encode_tmap_2d(&tm_dx, dx, (uint64_t)tokens, kN, kN * 2, 64, 64, 128));
    } else {
        tm_R = tm_Lt;
        tm_dx = tm_du;
    }
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(fused_bwd_dx_m64_kernel,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    BwdParams p;
    p.status = status;
    p.counters = counters;
    p.du = (__nv_bfloat16 *)du;
    p.dyp = (__nv_bfloat16 *)dyp;
    p.dy = (const __nv_bfloat16 *)dy;
    p.tokens = tokens;
    p.tiles = (int)tiles;
    // B1 gathers narrow rows (its TMA unit handles about one 16-byte row per 1.2 cycles) and transposes its
    // input: two thirds of the SMs (12 + 6 CTAs per group was the best of a sweep on 148 SMs)
    int b1 = both ? (sms * 12) / 148 : sms / 8;
    if (b1 < 1) b1 = 1;
    int b2 = both ? (sms - 8 * b1) / 8 : 0;
#ifdef MONARCH_TRACE
    if (const char *e = getenv("MONARCH_BWD_SPLIT2")) { if (both) sscanf(e, "%d,%d", &b1, &b2); }
#endif
    if (both && b2 < 1) b2 = 1;
    if (b1 > tiles) b1 = (int)tiles;
    if (b2 > tiles) b2 = (int)tiles;
    p.b1 = b1;
    p.b2 = b2;
    p.b3 = 0;
    p.want_dx = 1;
    p.need = kB1Arrivals;
    p.reset_at = kB1Arrivals + kB2Groups;
    p.u = nullptr;
    p.dL = p.dR = nullptr;
    p.trace = nullptr;
#ifdef MONARCH_TRACE
    if (const char *e = getenv("MONARCH_TRACE_PTR_BWD")) p.trace = (long long *)strtoull(e, nullptr, 0);
#endif
    fused_bwd_dx_m64_kernel<<<8 * b1 + 8 * b2, kThreads, kSmemBytes, s>>>(tm_dy3, tm_Lt, tm_R, tm_du, tm_dx, p);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}
}  // namespace

namespace {
// dW = (accumulate ? dW : 0) + part[0] + part[1] + ... in this order: the same bits every run
__global__ void reduce_partials_kernel(float4 *__restrict__ dW, const float4 *__restrict__ part, int count, int accumulate,
                                       int n4)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    float4 acc = accumulate ? dW[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < count; ++s) {
        const float4 v = part[(size_t)s * n4 + i];
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    dW[i] = acc;
}
}  // namespace

// dx, dL += , dR += in one launch (see the all-in-one kernel); u = u' in the forward exchange layout.
// partials != null (kBwdPartialBytes of scratch): the CTAs store their partial sums there and a second small launch adds
// them in a fixed order: dL, dR = (accumulate ? old : 0) + sums, bit-identical from run to run.
int fused_bwd_all_m64(const void *x, const void *dy, const void *L, const void *R, const void *u, void *dx,
                      void *du, void *dyp, float *dL, float *dR, unsigned *counters, unsigned *status,
                      int64_t tokens, cudaStream_t s, float *partials, int accumulate)
{
    using namespace tc;
    if (tokens == 0) return MONARCH_OK;
    const long long tiles = (tokens + 63) / 64;
    if (tiles * 4 > (long long)kBwdCounterBytes) return MONARCH_ERR_UNSUPPORTED;
    CUtensorMap tm_dy3, tm_Lt, tm_R, tm_du, tm_dx, tm_x;
    {
        const uint64_t dims[3] = {64, 64, (uint64_t)tokens}, strides[2] = {128, (uint64_t)kN * 2};
        const uint32_t box[3] = {8, 16, 64};
        MONARCH_TRY(encode_tmap_nd(&tm_dy3, dy, 2, 3, dims, strides, box));
        const uint64_t udims[3] = {128, 8, (uint64_t)tiles * 64}, ustrides[2] = {1024, 8192};
        const uint32_t ubox[3] = {128, 2, 4};
        MONARCH_TRY(encode_tmap_nd(&tm_du, du, 8, 3, udims, ustrides, ubox));
    }
    MONARCH_TRY(encode_tmap_2d(&tm_Lt, L, kN, kM, kM * 2, 64, 64, 128));
    MONARCH_TRY(encode_tmap_2d(&tm_R, R, kN, kM, kM * 2, 64, 64, 128));
    // dx == null: weight gradients only (the map is never used; it only has to be a valid one)
    MONARCH_TRY(encode_tmap_2d(&tm_dx, dx ? dx : x, (uint64_t)tokens, kN, kN * 2, 64, 64, 128));
    MONARCH_TRY(encode_tmap_2d(&tm_x, x, (uint64_t)tokens, kN, kN * 2, 64, 64, 128));
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(fused_bwd_all_m64_kernel,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    BwdParams p;
    p.status = status;
    p.counters = counters;
    p.du = (__nv_bfloat16 *)du;
    p.dyp = (__nv_bfloat16 *)dyp;
    p.dy = (const __nv_bfloat16 *)dy;
    p.u = (const __nv_bfloat16 *)u;
    p.dL = dL;
    p.dR = dR;
    p.want_dx = dx != nullptr;
    p.tokens = tokens;
    p.tiles = (int)tiles;
    // SM split: 8/7/7 CTAs per group (8 B1 groups, 8 B2R groups, 4 WL groups: all 148 SMs) was the best of a sweep
    // on 148 SMs; one CTA per group less of the first two kinds costs 2-10 %
    int b1 = (sms * 8) / 144, b2 = (sms * 7) / 144, b3 = (sms * 7) / 144;
    // weight gradients only: the B2R kind has half the work, 10/4/7 was the best of a sweep (132 against 140 us)
    if (dx == nullptr) { b1 = (sms * 10) / 144; b2 = (sms * 4) / 144; b3 = (sms * 7) / 144; }
#ifdef MONARCH_TRACE
    if (const char *e = getenv("MONARCH_BWD_SPLIT3")) sscanf(e, "%d,%d,%d", &b1, &b2, &b3);
#endif
    if (b1 < 1) b1 = 1;
    if (b2 < 1) b2 = 1;
    if (b3 < 1) b3 = 1;
    if (b1 > tiles) b1 = (int)tiles;
    if (b2 > tiles) b2 = (int)tiles;
    if (b3 > tiles) b3 = (int)tiles;
    if (8 * b1 + 8 * b2 + 4 * b3 > sms) return MONARCH_ERR_UNSUPPORTED;   // all CTAs must be co-resident
    if (partials != nullptr && (b2 > kBwdMaxPartials || b3 > kBwdMaxPartials)) return MONARCH_ERR_UNSUPPORTED;
    p.part_dR = partials;
    p.part_dL = partials ? partials + (size_t)kBwdMaxPartials * (kN * kM) : nullptr;
    // the gradients (or the slots of the partial sums) as [rows of 64 fp32] in boxes of 16 rows x 32 columns
    CUtensorMap tm_gL, tm_gR;
    {
        const uint64_t rows = (uint64_t)(partials ? kBwdMaxPartials : 1) * kN;
        const uint64_t dims[2] = {(uint64_t)kM, rows}, strides[1] = {(uint64_t)kM * sizeof(float)};
        const uint32_t box[2] = {32, 16};
        MONARCH_TRY(encode_tmap_nd(&tm_gL, partials ? p.part_dL : dL, 4, 2, dims, strides, box, 128));
        MONARCH_TRY(encode_tmap_nd(&tm_gR, partials ? p.part_dR : dR, 4, 2, dims, strides, box, 128));
    }
    p.b1 = b1;
    p.b2 = b2;
    p.b3 = b3;
    p.need = kB1Arrivals + 8 * kDypWarps;       // du from 16 store warps + P dy from 16 copy warps
    p.reset_at = p.need + 8 + 4;                // + 8 B2R groups + 4 WL groups
    p.trace = nullptr;
#ifdef MONARCH_TRACE
    if (const char *e = getenv("MONARCH_TRACE_PTR_BWD")) p.trace = (long long *)strtoull(e, nullptr, 0);
#endif
    fused_bwd_all_m64_kernel<<<8 * b1 + 8 * b2 + 4 * b3, kThreads, kSmemBytes, s>>>(tm_dy3, tm_Lt, tm_R, tm_du, tm_dx,
                                                                                 tm_x, tm_gL, tm_gR, p);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    if (partials != nullptr) {
        // a CTA of a group takes tiles first, first + step, ...: CTAs beyond the tile count have no partial sums
        const int n4 = kN * kM / 4;
        reduce_partials_kernel<<<(n4 + 255) / 256, 256, 0, s>>>((float4 *)dR, (const float4 *)p.part_dR, b2, accumulate, n4);
        reduce_partials_kernel<<<(n4 + 255) / 256, 256, 0, s>>>((float4 *)dL, (const float4 *)p.part_dL, b3, accumulate, n4);
        note_launch(2);
        MONARCH_CUDA_TRY(cudaGetLastError());
    }
    return MONARCH_OK;
}

int fused_bwd_dx_m64(const void *dy, const void *L, const void *R, void *dx, int64_t tokens, void *ws,
                     cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    return launch_bwd_m64(dy, L, R, dx, (char *)ws + MONARCH_STATUS_BYTES + kBwdCounterBytes, nullptr,
                          (unsigned *)((char *)ws + MONARCH_STATUS_BYTES), (unsigned *)ws, tokens, s);
}

int fused_bwd_dx_m64_keep(const void *dy, const void *L, const void *R, void *dx, void *du, void *dyp,
                          unsigned *counters, unsigned *status, int64_t tokens, cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    return launch_bwd_m64(dy, L, R, dx, du, dyp, counters, status, tokens, s);
}

int fused_bwd_m64_stage1(const void *dy, const void *L, void *du, void *dyp, int64_t tokens,
                         unsigned *status, cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    return launch_bwd_m64(dy, L, nullptr, nullptr, du, dyp, nullptr, status, tokens, s);
}

}  // namespace monarch
