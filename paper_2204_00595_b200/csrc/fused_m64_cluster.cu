// Fused forward y = P L P^T R x for m = 64 (n = 4096), bf16, on clusters of four CTAs: the permuted intermediate
// of Section 3.3 (steps 1-3) never leaves the cluster's shared memory.
//
// A cluster takes a 64-token tile.  CTA c of the cluster owns the 16 stage-1 blocks k = 16c .. 16c+15 and the 16
// stage-2 blocks j = 16c .. 16c+15.
//   stage 1   D_k[j][t] = sum_i R[k][j][i] x[t][k*64+i]      A = R_k (rows j), B = the 64 x 64 tile of x (rows t),
//             tcgen05.mma M = 64, N = 64 tokens; 16 accumulators fill TMEM (two 16-lane halves x 512 columns).
//   exchange  row j of D_k is 64 tokens = 128 bytes; it is row k of the stage-2 operand of block j, which lives in
//             the shared memory of CTA j / 16.  The epilogue thread of row j (warp j / 16: a warp has ONE
//             destination) writes it there with 16-byte asynchronous distributed-shared-memory stores that count
//             their bytes on the destination's barrier - already in the 128-byte-swizzled MN-major operand layout
//             (rows = k, tokens along the row).  This is the inner P^T of Def. 3.1.
//   stage 2   D_j[l][t] = sum_k L[j][l][k] u'_j[k][t]          A = L_j (rows l), B = the received slab (MN-major).
//   output    thread (row l) finds the 16 blocks j of its CTA side by side in TMEM; y[t][l*64+16c .. +16) leaves as
//             32-byte rows of 3-D TMA boxes (the load/store units manage 12 B/clk on such pieces, the TMA unit 27):
//             the outer P of step 3.
// Weights are not resident (16 + 16 blocks of 8 KB per CTA and tile = 256 KB would leave no room for the operand
// slab): they stream from L2 through a ring as linear bulk copies of blocks that a small kernel has put into the
// swizzled operand image once per call (linear copies run at 72 B/clk per SM, tiled TMA copies at 33; measured).
// Per tile and CTA: 128 KB of x (tiled TMA), 256 KB of weights (L2), 96 KB through distributed shared memory
// (16 B/clk measured: the longest leg), 128 KB of y.
// Every wait is bounded; a cluster leaves together.
#include <cstdlib>

#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

constexpr int kM = 64, kN = kM * kM;
constexpr int kCluster = 4, kBlk = kM / kCluster;            // blocks per CTA and stage
constexpr int kTile = 64;                                    // tokens per tile
constexpr int kBlockBytes = kM * kM * 2;                     // 8 KB: one weight block, one x tile, one operand slab
constexpr int kWSlots = 4, kXSlots = 4;
constexpr int kThreads = 8 * 32;                             // warps 0-3 epilogue, 4 weight loader, 5 x loader, 6 MMA, 7 helper
constexpr int kWarpStageBytes = 8192;                        // per epilogue warp: two 4 KB buffers
constexpr int kSmem = kBlk * kBlockBytes + kWSlots * kBlockBytes + kXSlots * kBlockBytes + 4 * kWarpStageBytes + 1024;
constexpr uint32_t kRemoteBytes = (kCluster - 1) * kBlk * kBlk * 128;   // what the other three CTAs send per tile

struct ClusterParams {
    unsigned *status;
    const char *Rimg, *Limg;          // weight blocks in the swizzled operand image
    long long tokens;
    int tiles, nclusters;
    long long *trace;                 // debug builds: per-CTA cycle sums, else null
};

#ifdef MONARCH_TRACE
#define CT0() const long long ct0_ = clock64()
#define CACC(v) v += clock64() - ct0_
#define COUT(site, v) do { if (p.trace) p.trace[blockIdx.x * 16 + (site)] = (v); } while (0)
#else
#define CT0() do { } while (0)
#define CACC(v) do { } while (0)
#define COUT(site, v) do { } while (0)
#endif

struct Bars {
    uint64_t w_full[kWSlots], w_empty[kWSlots];
    uint64_t x_full[kXSlots], x_empty[kXSlots];
    uint64_t s1_full[4];              // stage-1 accumulators of a group of four blocks are complete
    uint64_t s2_full;                 // all stage-2 accumulators of the tile are complete
    uint64_t tm_free;                 // the stage-2 epilogue has read all of TMEM
    uint64_t u_full;                  // the operand slabs of this CTA are complete (remote bytes + own rows)
    uint64_t u_done;                  // this CTA's stage-2 MMAs have read the slabs
    uint64_t u_free;                  // ... in all four CTAs: the slabs of the whole cluster may be overwritten
};

__device__ __forceinline__ void bulk_load_linear(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
                 "r"(bytes), "r"(bar)
                 : "memory");
}
// 16-byte store into another CTA's shared memory whose bytes are counted on that CTA's barrier
__device__ __forceinline__ void st_async_v4(uint32_t cluster_addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t cluster_bar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(cluster_addr),
                 "r"(a), "r"(b), "r"(c), "r"(d), "r"(cluster_bar)
                 : "memory");
}

__global__ void __cluster_dims__(kCluster, 1, 1) __launch_bounds__(kThreads, 1)
fused_fwd_m64_cluster_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_y, const ClusterParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) Bars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead_s;

    const uint32_t U0 = (smem_u32(smem_raw) + 1023u) & ~1023u;          // 16 slabs [k 64 rows][64 t]
    const uint32_t wring0 = U0 + kBlk * kBlockBytes;
    const uint32_t xring0 = wring0 + kWSlots * kBlockBytes;
    const uint32_t stage0 = xring0 + kXSlots * kBlockBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t c = cluster_ctarank();
    const int cid = (int)blockIdx.x / kCluster;
    volatile int *dead = &dead_s;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kWSlots; ++s) {
            mbar_init(smem_u32(&bars.w_full[s]), 1);
            mbar_init(smem_u32(&bars.w_empty[s]), 1);
        }
        for (int s = 0; s < kXSlots; ++s) {
            mbar_init(smem_u32(&bars.x_full[s]), 1);
            mbar_init(smem_u32(&bars.x_empty[s]), 1);
        }
        for (int g = 0; g < 4; ++g) mbar_init(smem_u32(&bars.s1_full[g]), 1);
        mbar_init(smem_u32(&bars.s2_full), 1);
        mbar_init(smem_u32(&bars.tm_free), 4);
        mbar_init(smem_u32(&bars.u_full), 5);                 // the expect_tx arrival + the four epilogue warps (stage-1 reads done)
        mbar_init(smem_u32(&bars.u_done), 1);
        mbar_init(smem_u32(&bars.u_free), kCluster);
        fence_mbar_init();
        dead_s = 0;
        tma_prefetch_desc(&tm_x); tma_prefetch_desc(&tm_y);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_arrive_release();                                  // every CTA's barriers exist before any remote access
    cluster_wait_acquire();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    const int nt = cid < p.tiles ? (p.tiles - cid + p.nclusters - 1) / p.nclusters : 0;   // tiles of this cluster
    const uint32_t wf0 = smem_u32(bars.w_full), we0 = smem_u32(bars.w_empty);
    const uint32_t xf0 = smem_u32(bars.x_full), xe0 = smem_u32(bars.x_empty);
    const uint32_t s1f0 = smem_u32(bars.s1_full), s2f = smem_u32(&bars.s2_full), tmfree = smem_u32(&bars.tm_free);
    const uint32_t ufull = smem_u32(&bars.u_full), udone = smem_u32(&bars.u_done), ufree = smem_u32(&bars.u_free);

    if (warp == 4) {
        // ------------------------------------------------------------ weight loader: R blocks, then L blocks, per tile
        if (lane == 0) {
            uint32_t n = 0;
            bool ok = true;
            for (int it = 0; ok && it < nt; ++it) {
#pragma unroll 1
                for (int bq = 0; bq < 2 * kBlk; ++bq, ++n) {
                    const uint32_t s = n % kWSlots;
                    if (!mbar_wait(we0 + s * 8, ((n / kWSlots) & 1) ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
                    const char *src = (bq < kBlk ? p.Rimg + (size_t)(c * kBlk + bq) * kBlockBytes
                                                 : p.Limg + (size_t)(c * kBlk + bq - kBlk) * kBlockBytes);
                    mbar_expect_tx(wf0 + s * 8, kBlockBytes);
                    bulk_load_linear(wring0 + s * kBlockBytes, src, kBlockBytes, wf0 + s * 8);
                }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ x loader: the 16 tiles x[tile][k*64 .. +64) of this CTA
        if (lane == 0) {
            uint32_t n = 0;
            bool ok = true;
            for (int it = 0; ok && it < nt; ++it) {
                const int tile = cid + it * p.nclusters;
#pragma unroll 1
                for (int kl = 0; kl < kBlk; ++kl, ++n) {
                    const uint32_t s = n % kXSlots;
                    if (!mbar_wait(xe0 + s * 8, ((n / kXSlots) & 1) ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
                    mbar_expect_tx(xf0 + s * 8, kBlockBytes);
                    tma_load_2d(xring0 + s * kBlockBytes, &tm_x, (int)(c * kBlk + kl) * kM, tile * kTile, xf0 + s * 8);
                }
            }
        }
    } else if (warp == 6) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc1 = make_idesc_bf16(64, 64, 0, 0), idesc2 = make_idesc_bf16(64, 64, 0, 1);
            const uint64_t dK = make_smem_desc(0, 16, 1024, kSwizzle128);       // K-major, 128-byte rows
            const uint64_t dMN = make_smem_desc(0, 8192, 1024, kSwizzle128);    // MN-major, one 64-wide atom
            uint32_t nw = 0, nx = 0;
            bool ok = true;
            [[maybe_unused]] long long wt = 0, wop = 0, wu = 0, wl = 0;
            [[maybe_unused]] const long long tm0 = clock64();
            for (int it = 0; ok && it < nt; ++it) {
                // ---- stage 1: block kl -> lane half kl & 1, columns (kl >> 1) * 64
                { CT0(); if (!mbar_wait(tmfree, (it & 1) ^ 1, p.status, dead, kErrTmemWait)) break; CACC(wt); }
                tc_fence_after();
#pragma unroll 1
                for (int kl = 0; kl < kBlk; ++kl, ++nw, ++nx) {
                    const uint32_t ws = nw % kWSlots, xs = nx % kXSlots;
                    { CT0(); if (!mbar_wait(wf0 + ws * 8, (nw / kWSlots) & 1, p.status, dead, kErrTmaWait)) { ok = false; break; }
                    if (!mbar_wait(xf0 + xs * 8, (nx / kXSlots) & 1, p.status, dead, kErrTmaWait)) { ok = false; break; } CACC(wop); }
                    tc_fence_after();
                    const uint64_t ad = dK | (uint64_t)((wring0 + ws * kBlockBytes) >> 4);
                    const uint64_t bd = dK | (uint64_t)((xring0 + xs * kBlockBytes) >> 4);
                    const uint32_t d = tmem_base + ((uint32_t)((kl & 1) * 16) << 16) + (kl >> 1) * 64;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) mma_f16_ss(d, ad + 2 * ks, bd + 2 * ks, idesc1, ks != 0);
                    mma_commit(we0 + ws * 8);
                    mma_commit(xe0 + xs * 8);
                    if ((kl & 3) == 3) mma_commit(s1f0 + (kl >> 2) * 8);
                }
                if (!ok) break;
                // ---- stage 2: all four CTAs' rows have landed; block jl -> lane half jl >> 3, columns (jl & 7) * 64
                { CT0(); if (!mbar_wait<true>(ufull, it & 1, p.status, dead, kErrPeerWait)) break; CACC(wu); }
                fence_proxy_async_smem();
                tc_fence_after();
#pragma unroll 1
                for (int jl = 0; jl < kBlk; ++jl, ++nw) {
                    const uint32_t ws = nw % kWSlots;
                    { CT0(); if (!mbar_wait(wf0 + ws * 8, (nw / kWSlots) & 1, p.status, dead, kErrTmaWait)) { ok = false; break; } CACC(wl); }
                    tc_fence_after();
                    const uint64_t ad = dK | (uint64_t)((wring0 + ws * kBlockBytes) >> 4);
                    const uint64_t bd = dMN | (uint64_t)((U0 + jl * kBlockBytes) >> 4);
                    const uint32_t d = tmem_base + ((uint32_t)((jl >> 3) * 16) << 16) + (jl & 7) * 64;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) mma_f16_ss(d, ad + 2 * ks, bd + 128 * ks, idesc2, ks != 0);
                    mma_commit(we0 + ws * 8);
                }
                if (!ok) break;
                mma_commit(s2f);
                mma_commit(udone);
            }
            COUT(0, wt); COUT(1, wop); COUT(2, wu); COUT(3, wl); COUT(4, clock64() - tm0);
        }
    } else if (warp == 7) {
        // ------------------------------------------------------------ helper: announces the bytes the slabs expect,
        // and tells the whole cluster when this CTA's stage 2 has read them
        if (lane == 0) {
            for (int it = 0; it < nt; ++it) {
                mbar_expect_tx(ufull, kRemoteBytes);
                if (!mbar_wait(udone, it & 1, p.status, dead, kErrMmaWait)) break;
                for (uint32_t d = 0; d < kCluster; ++d) mbar_arrive_remote(map_to_cta(ufree, d));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogues (warps 0-3 = TMEM lane quarters)
        const int q = warp, hl = lane >> 4;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t stg = stage0 + warp * kWarpStageBytes;             // this warp's 8 KB: two 4 KB buffers
        // stage-1 rows of this warp (j = 16 q .. 16 q + 15) all go to CTA q
        const uint32_t dstU = map_to_cta(U0, (uint32_t)q);
        const uint32_t dstBar = map_to_cta(ufull, (uint32_t)q);
        const bool local = (uint32_t)q == c;
        bool ok = true;
        [[maybe_unused]] long long wfree = 0, ws1 = 0, ws2 = 0, b1 = 0, b2 = 0;
        for (int it = 0; ok && it < nt; ++it) {
            const int tile = cid + it * p.nclusters;
            // the previous tile's slabs have been read by stage 2 in every CTA of the cluster
            { CT0(); if (!mbar_wait<true>(ufree, (it & 1) ^ 1, p.status, dead, kErrPeerWait)) break; CACC(wfree); }
            [[maybe_unused]] const long long e1 = clock64();
#pragma unroll 1
            for (int g = 0; g < 4 && ok; ++g) {
                { CT0(); if (!mbar_wait(s1f0 + g * 8, it & 1, p.status, dead, kErrMmaWait)) { ok = false; break; } CACC(ws1); }
                tc_fence_after();
#pragma unroll 1
                for (int e = 0; e < 2; ++e) {
                    // this lane half holds the blocks with kl & 1 == hl: row r = 16 hl + (j & 15) of the 4 KB buffer
                    const int kl = g * 4 + e * 2 + hl;
                    const uint32_t buf = stg + (e & 1) * 4096;
                    const int r = lane;
                    uint32_t v[4][16];
#pragma unroll
                    for (int i = 0; i < 4; ++i) tmem_ld16(lane_base + (kl >> 1) * 64 + i * 16, v[i]);
                    tmem_ld_wait();
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch) {
                        const uint32_t *w = &v[ch >> 1][(ch & 1) * 8];
                        const uint32_t o0 = pack_bf16(__uint_as_float(w[0]), __uint_as_float(w[1]));
                        const uint32_t o1 = pack_bf16(__uint_as_float(w[2]), __uint_as_float(w[3]));
                        const uint32_t o2 = pack_bf16(__uint_as_float(w[4]), __uint_as_float(w[5]));
                        const uint32_t o3 = pack_bf16(__uint_as_float(w[6]), __uint_as_float(w[7]));
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(buf + r * 128 + ((ch ^ (r & 7)) << 4)),
                                     "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                    }
                    __syncwarp();
                    // out again eight lanes per 128-byte row (distributed shared memory moves 16 B/clk with whole rows
                    // per instruction, half of that with one 16-byte piece per lane and row): row rr of the buffer is
                    // row k of slab j & 15 in CTA q, its chunks XORed with k % 8
                    const int ch = lane & 7;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int rr = i * 4 + (lane >> 3);
                        const int k = (int)c * kBlk + g * 4 + e * 2 + (rr >> 4);
                        uint32_t o0, o1, o2, o3;
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(o0), "=r"(o1), "=r"(o2), "=r"(o3)
                                     : "r"(buf + rr * 128 + ((ch ^ (rr & 7)) << 4)) : "memory");
                        const uint32_t a = dstU + (rr & 15) * kBlockBytes + k * 128 + ((ch ^ (k & 7)) << 4);
                        if (local) st_cluster_v4(a, o0, o1, o2, o3);
                        else st_async_v4(a, o0, o1, o2, o3, dstBar);
                    }
                }
            }
            if (!ok) break;
            // this warp has read its stage-1 accumulators (stage 2 overwrites them) and, if it wrote rows into its own
            // CTA with ordinary stores, these must be visible to the tensor cores' reads: count the warp on the slab barrier
            tc_fence_before();
            if (local) fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(ufull);
            // ---- stage 2: row l = 16 q + (lane & 15), blocks jl = 8 hl .. 8 hl + 7 side by side -> 16 bytes of y per
            // token; eight tokens at a time through this warp's buffers as [t 8][l 4][16 j] boxes per group of four rows
            b1 += clock64() - e1;
            { CT0(); if (!mbar_wait(s2f, it & 1, p.status, dead, kErrMmaWait)) break; CACC(ws2); }
            tc_fence_after();
            [[maybe_unused]] const long long e2 = clock64();
            const int lc = (lane & 15) >> 2, li = lane & 3;
#pragma unroll 1
            for (int pc = 0; pc < kTile / 8; ++pc) {
                const uint32_t buf = stg + (pc & 1) * 4096;
                uint32_t v[8][8];
#pragma unroll
                for (int a = 0; a < 8; ++a) tmem_ld8(lane_base + a * 64 + pc * 8, v[a]);
                tmem_ld_wait();
                if (pc + 1 == kTile / 8) {
                    // TMEM is in registers: stage 1 of the next tile may overwrite it
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tmfree);
                }
                // the stores issued from this buffer two pieces ago have read it
                if (lane < 4) tma_store_wait_read<1>();
                __syncwarp();
#pragma unroll
                for (int tt = 0; tt < 8; ++tt) {
                    const uint32_t o0 = pack_bf16(__uint_as_float(v[0][tt]), __uint_as_float(v[1][tt]));
                    const uint32_t o1 = pack_bf16(__uint_as_float(v[2][tt]), __uint_as_float(v[3][tt]));
                    const uint32_t o2 = pack_bf16(__uint_as_float(v[4][tt]), __uint_as_float(v[5][tt]));
                    const uint32_t o3 = pack_bf16(__uint_as_float(v[6][tt]), __uint_as_float(v[7][tt]));
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(buf + lc * 1024 + tt * 128 + li * 32 + hl * 16),
                                 "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane < 4) {
                    // y as [t][l][j]: box 16 j x 4 l x 8 t; tokens past the last one are clipped
                    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(&tm_y),
                                 "r"(buf + lane * 1024), "r"((int)c * 16), "r"(q * 16 + lane * 4), "r"(tile * kTile + pc * 8) : "memory");
                    tma_store_commit();
                }
            }
            // the buffers go back to stage 1
            if (lane < 4) tma_store_wait_read<0>();
            __syncwarp();
            b2 += clock64() - e2;
        }
        if (lane < 4) tma_store_wait_all<0>();
        if (threadIdx.x == 0) { COUT(5, wfree); COUT(6, ws1); COUT(7, ws2); COUT(8, b1); COUT(9, b2); }
    }

    // remote stores and arrivals target this CTA until every CTA of the cluster is done: leave together
    tc_fence_before();
    __syncthreads();
    cluster_arrive_release();
    cluster_wait_acquire();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

// Weight blocks [block][64 rows][64 columns] -> the same with the eight 16-byte chunks of every row stored at
// (chunk XOR row % 8): the 128-byte-swizzled K-major operand image, so that a block is one linear copy away from
// shared memory.
__global__ void weight_image_kernel(const uint4 *__restrict__ W, uint4 *__restrict__ out, int chunks)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= chunks) return;
    const int row = (i >> 3) & 63, ch = i & 7;
    out[(i & ~7) | (ch ^ (row & 7))] = W[i];
}

}  // namespace
}  // namespace tc

// Workspace use: [status][64 KB unused][R image 512 KB][L image 512 KB] (inside the area of the exchange buffer of the
// other m = 64 forward kernels).  Returns MONARCH_ERR_UNSUPPORTED when no cluster of four fits the device.
int fused_fwd_m64_cluster(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws, cudaStream_t s)
{
    using namespace tc;
    if (tokens == 0) return MONARCH_OK;
    const long long tiles = (tokens + kTile - 1) / kTile;
    if (tiles > (1 << 24)) return MONARCH_ERR_UNSUPPORTED;
    static PerDeviceCache max_clusters_cache;
    int max_clusters = max_clusters_cache.get();
    if (max_clusters < 0) {
        MONARCH_CUDA_TRY(cudaFuncSetAttribute(fused_fwd_m64_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem));
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(kCluster, 1, 1);
        cfg.blockDim = dim3(kThreads, 1, 1);
        cfg.dynamicSmemBytes = kSmem;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = kCluster; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, fused_fwd_m64_cluster_kernel, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
        max_clusters = n;
        max_clusters_cache.set(n);
    }
    if (max_clusters < 1) return MONARCH_ERR_UNSUPPORTED;
    char *Rimg = (char *)ws + MONARCH_STATUS_BYTES + 65536, *Limg = Rimg + (size_t)kN * kM * 2;
    const int chunks = kN * kM * 2 / 16;
    weight_image_kernel<<<(chunks + 255) / 256, 256, 0, s>>>((const uint4 *)R, (uint4 *)Rimg, chunks);
    weight_image_kernel<<<(chunks + 255) / 256, 256, 0, s>>>((const uint4 *)L, (uint4 *)Limg, chunks);
    note_launch(2);
    CUtensorMap tm_x, tm_y;
    MONARCH_TRY(encode_tmap_2d(&tm_x, x, (uint64_t)tokens, kN, kN * 2, kTile, 64, 128));
    {
        const uint64_t ydims[3] = {64, 64, (uint64_t)tokens}, ystrides[2] = {128, (uint64_t)kN * 2};     // [t][l][j]
        const uint32_t ybox[3] = {16, 4, 8};
        MONARCH_TRY(encode_tmap_nd(&tm_y, y, 2, 3, ydims, ystrides, ybox));
    }
    ClusterParams p;
    p.status = (unsigned *)ws;
    p.Rimg = Rimg;
    p.Limg = Limg;
    p.tokens = tokens;
    p.tiles = (int)tiles;
    p.nclusters = (int)(tiles < max_clusters ? tiles : max_clusters);
    p.trace = nullptr;
#ifdef MONARCH_TRACE
    if (const char *e = getenv("MONARCH_TRACE_PTR")) p.trace = (long long *)strtoull(e, nullptr, 0);
#endif
    fused_fwd_m64_cluster_kernel<<<kCluster * p.nclusters, kThreads, kSmem, s>>>(tm_x, tm_y, p);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

}  // namespace monarch
