// m = 128 (n = 16384), bf16: the Monarch multiply and its adjoints as chains of block GEMMs whose stride
// permutations cost nothing on chip.
//
// The permutation between the two stages of Section 3.3 (steps 1-3) moves 2-byte elements: u'[t][j][k] = u[t][k][j].
// With 128 x 128 blocks neither the accumulators of 16 blocks (for 32-byte pieces) nor a token tile of u (32 KB per
// token) fit an SM, so the permuted intermediate cannot be assembled on chip.  What can be chosen freely is which
// index of an intermediate is contiguous in memory: the tensor cores read an operand either with its contraction
// index contiguous ("K-major") or with its row/column index contiguous ("MN-major").  All intermediates here are
// stored TOKEN-INNERMOST in tiles of 128 tokens and CONSUMER-CONTIGUOUS: every intermediate is written by 128
// producer blocks p and read by 128 consumer blocks c (every consumer needs one 128 x 128 slab made of one row of
// every producer's result), and lives as
//     [tile][c][half h][p][64 tokens]      (a 128-byte row = tokens 64h .. 64h+63 of row c of producer p's result)
// with the eight 16-byte chunks of a row stored at position (chunk XOR p % 8).  A consumer's slab [c] is then 32 KB
// contiguous and is, byte for byte, the 128-byte-swizzled shared-memory image of a tensor-core operand with rows p:
// ONE linear bulk copy fetches it (linear copies run at 72 B/clk per SM, tiled TMA copies of 128-byte rows at 33;
// measured), read MN-major (tokens as the row/column index) by the block products and K-major (tokens as the
// contraction index) by the token reductions.  A producer writes 128-byte pieces 32 KB apart.
//     u'  (c = j, p = k)  rows j of D_k[j][t] = R_k x_k        -> operand of stage 2, block j
//     w'  (c = l, p = j)  rows l of D_j[l][t] = L_j u'_j       -> plane l, transposed through shared memory
//                         (ldmatrix.trans / stmatrix) into y[t][l*128 + j]
// So the inner permutation of Def. 3.1 is the choice of where a row goes, the outer one a plane transpose, and every
// global access of the chain is a full 128-byte line.  The adjoints reverse the chain (dy transposed into
// dw' (c = j, p = l), du'[k][t] = L_j^T dw'_j stored as du' (c = k, p = j), dx = du'_k^T R_k), and because the token
// index is contiguous the same slabs are K-major operands of the token reductions dL_j = dw'_j u'_j^T and
// dR_k = du'_k x_k, which ride along in the same kernels with their accumulators resident in TMEM for all tiles of a
// block (one writer per block: deterministic sums).
//
// L2 management: an intermediate (134 MB at 4096 tokens) is larger than what L2 keeps, and the backward launches are
// bound by DRAM, so (i) every load of data that nothing reads again carries an evict-first policy, (ii) the pieces of an
// intermediate are stored evict-last and the next launch walks the tiles in the opposite direction, (iii) a consumed
// slab is dropped from L2 without a write-back (discard.global.L2) - dead dirty lines never reach DRAM.
//
// One kernel template serves all block products: persistent CTAs, the 32 KB weight block resident, token operands
// through a TMA ring, tcgen05.mma 128 x 128 x 16 with two accumulator buffers in TMEM, epilogue through swizzled
// staging tiles and TMA stores.
#include <atomic>
#include <cstdlib>
#include <utility>

#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

// Host-side fault injection for the test of the bounded waits: the next plane-transpose launch leaves out the load of
// this item (neither announced nor copied), so its consumers wait for bytes that never come.  -1 = none.
std::atomic<long long> g_skip_load{-1};
// forward pass in one persistent launch (default) or in three launches (comparison runs: MONARCH_CHAIN_SPLIT set)
bool chain_fused_enabled()
{
    static const bool on = getenv("MONARCH_CHAIN_SPLIT") == nullptr;
    return on;
}

constexpr int kB = 128;                      // block size m
constexpr int kOpBytes = 32768;              // one 128 x 128 bf16 operand: two boxes of [128 rows][64 columns]
constexpr int kHalfBytes = 16384;
constexpr int kThreads = 7 * 32;             // warps 0-3 epilogue, 4 loader, 5 MMA, 6 drops consumed slabs from L2
constexpr int kStagingBytes = 2 * kHalfBytes;

enum { kLdX = 0, kLdC = 1 };                 // token-major tensor (tiled TMA); consumer slab of an intermediate (linear)
enum { kStX = 0, kStP = 1 };                 // token-major tensor; producer pieces of an intermediate

struct ChainParams {
    unsigned *status;
    float *dW;                               // token-reduction output [block][128][128]
    int overwrite;                           // 1: dW = sums, 0: dW += sums
    const char *t0_base, *t1_base;           // intermediates read as consumer slabs (kLdC)
    int ntiles;                              // 128-token tiles
    int nblk;                                // blocks (128)
    int reverse;                             // walk the tiles from the last to the first: what the previous launch of
                                             // the chain wrote last is still in L2
    int discard_t0;                          // the T0 slabs are dead once read (dw', du'; not u', which the backward call reads)
};

struct ChainBars {
    uint64_t full[4], empty[4];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t w_full[2], w_empty[2];
    uint64_t wg_full, wg_empty;
};

// Programmatic dependent launch: a kernel of the chain lets its successor start as SMs become free (barrier set-up, TMEM
// allocation and the weight load overlap this kernel's tail); the successor waits here, once per thread, before it
// touches anything the chain wrote.  Both are no-ops in a launch without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void tma_store_5d(const CUtensorMap *m, uint32_t src, int c0, int c1, int c2, int c3, int c4)
{
    asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5, %6}], [%1];" ::"l"(m), "r"(src),
                 "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
                 : "memory");
}
__device__ __forceinline__ void bulk_load_linear(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src),
                 "r"(bytes), "r"(bar)
                 : "memory");
}

// Data with no further use in this launch (an intermediate's slab at its one read, the input, the output) is marked
// evict-first in L2, so that it does not push out the rows that are read back a few steps after they were written.
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_2d_last_use(uint32_t dst, const CUtensorMap *m, int x, int y, uint32_t bar, uint64_t pol)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%3, %4}], [%2], %5;" ::"r"(dst),
        "l"(m), "r"(bar), "r"(x), "r"(y), "l"(pol)
        : "memory");
}
__device__ __forceinline__ uint64_t l2_evict_last_policy()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_store_5d_keep(const CUtensorMap *m, uint32_t src, int c0, int c1, int c2, int c3, int c4, uint64_t pol)
{
    asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3, %4, %5, %6}], [%1], %7;" ::"l"(m),
                 "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "l"(pol)
                 : "memory");
}
__device__ __forceinline__ void tma_store_2d_stream(const CUtensorMap *m, uint32_t src, int x, int y, uint64_t pol)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;" ::"l"(m),
                 "r"(src), "r"(x), "r"(y), "l"(pol)
                 : "memory");
}
// a 32-column x 128-row fp32 piece of a weight gradient block: stored, or added to what is there (one writer per element)
__device__ __forceinline__ void tma_store_2d_plain(const CUtensorMap *m, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(m), "r"(src), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap *m, uint32_t src, int x, int y)
{
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(m), "r"(src),
                 "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void bulk_load_linear_last_use(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint64_t pol)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar), "l"(pol)
                 : "memory");
}

// An intermediate's slab is read exactly once, by one CTA.  Once its copy has landed in shared memory the 256 lines are
// dropped from L2 without a write-back (what is still dirty there would otherwise go to DRAM for nothing); the values
// at those addresses are undefined until the next call writes them again.  One warp: 8 lines per lane.
__device__ __forceinline__ void discard_slab(const char *slab, int lane)
{
#pragma unroll
    for (int i = 0; i < 8; ++i) asm volatile("discard.global.L2 [%0], 128;" ::"l"(slab + (i * 32 + lane) * 128) : "memory");
}

// Load one 128 x 128 operand of block `blk`, tile `tile`: two 64-column boxes of a token-major tensor, or the
// consumer slab [tile][blk] of an intermediate (already the swizzled image).
template <int KIND>
__device__ __forceinline__ void load_operand(uint32_t dst, const CUtensorMap *m, const char *base, int blk, int tile, uint32_t bar)
{
    if (KIND == kLdX) {
        tma_load_2d(dst, m, blk * kB, tile * 128, bar);
        tma_load_2d(dst + kHalfBytes, m, blk * kB + 64, tile * 128, bar);
    } else {
        bulk_load_linear(dst, base + ((size_t)tile * kB + blk) * kOpBytes, kOpBytes, bar);
    }
}
// the same for an operand that is not read again by this launch or the next ones of the chain
template <int KIND>
__device__ __forceinline__ void load_operand_last_use(uint32_t dst, const CUtensorMap *m, const char *base, int blk, int tile,
                                                      uint32_t bar, uint64_t pol)
{
    if (KIND == kLdX) {
        tma_load_2d_last_use(dst, m, blk * kB, tile * 128, bar, pol);
        tma_load_2d_last_use(dst + kHalfBytes, m, blk * kB + 64, tile * 128, bar, pol);
    } else {
        bulk_load_linear_last_use(dst, base + ((size_t)tile * kB + blk) * kOpBytes, kOpBytes, bar, pol);
    }
}

// Descriptor of K-step s (16 of the contraction index) of an operand tile: with the contraction index along the
// 128-byte rows (K-major: four steps per box) or down the rows (MN-major: 16 rows = 2 KB per step, the two boxes
// side by side along the row/column index).
__device__ __forceinline__ uint64_t op_desc(uint32_t base, bool mn, int s)
{
    return mn ? make_smem_desc(base + s * 2048, kHalfBytes, 1024, kSwizzle128)
              : make_smem_desc(base + (s >> 2) * kHalfBytes + (s & 3) * 32, 16, 1024, kSwizzle128);
}

// D = A B^T per (block, tile).  W_IS_A: the weight block is the A operand (rows of D = weight rows or columns,
// columns of D = tokens) else the token operand T0 is A (rows of D = tokens).  *_MN: operand read MN-major.
// WG: additionally dW[blk] += T0 (rows as M, tokens as K) x T1 (T1_MN ? token-major natural tensor : [..][t]).
// MAIN = false drops the main product (weight gradients only).
template <int T0_LD, bool W_IS_A, bool W_MN, bool T0_MN, int ST, bool WG, int T1_LD, bool T1_MN, bool MAIN, int SLOTS>
__global__ void __launch_bounds__(kThreads, 1)
chain_gemm_kernel(const __grid_constant__ CUtensorMap tm_t0, const __grid_constant__ CUtensorMap tm_t1,
                  const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_out,
                  const __grid_constant__ CUtensorMap tm_dw, const ChainParams p)
{
    constexpr int kSlotBytes = WG ? 2 * kOpBytes : kOpBytes;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) ChainBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead_s;

    const uint32_t w0 = (smem_u32(smem_raw) + 1023u) & ~1023u;          // two weight buffers
    const uint32_t ring0 = w0 + 2 * kOpBytes;
    const uint32_t staging0 = ring0 + SLOTS * kSlotBytes;                // two 16 KB staging tiles
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *dead = &dead_s;

    if (threadIdx.x == 0) {
        for (int s = 0; s < SLOTS; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), T0_LD == kLdC ? 2 : 1);      // the MMAs, and the warp that drops the slab
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&bars.acc_full[a]), 1);
            mbar_init(smem_u32(&bars.acc_empty[a]), 4);
            mbar_init(smem_u32(&bars.w_full[a]), 1);
            mbar_init(smem_u32(&bars.w_empty[a]), 1);
        }
        mbar_init(smem_u32(&bars.wg_full), 1);
        mbar_init(smem_u32(&bars.wg_empty), 4);
        fence_mbar_init();
        dead_s = 0;
        tma_prefetch_desc(&tm_t0); tma_prefetch_desc(&tm_w);
        if (MAIN) tma_prefetch_desc(&tm_out);
        if (WG) { tma_prefetch_desc(&tm_t1); tma_prefetch_desc(&tm_dw); }
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    if (!(warp == 4 && lane == 0)) pdl_wait();          // the loader waits after it has asked for its first weight block

    // items = (block, tile), block-major.  With a token reduction a CTA owns whole blocks (its accumulator lives in
    // TMEM across the tiles of a block); otherwise the items are cut into equal contiguous runs.
    long long i0, i1;
    if (WG) {
        i0 = (long long)p.nblk * blockIdx.x / gridDim.x * p.ntiles;
        i1 = (long long)p.nblk * (blockIdx.x + 1) / gridDim.x * p.ntiles;
    } else {
        const long long total = (long long)p.nblk * p.ntiles;
        i0 = total * blockIdx.x / gridDim.x;
        i1 = total * (blockIdx.x + 1) / gridDim.x;
    }
    const uint32_t full0 = smem_u32(bars.full), empty0 = smem_u32(bars.empty);
    const uint32_t accf0 = smem_u32(bars.acc_full), acce0 = smem_u32(bars.acc_empty);
    const uint32_t wf0 = smem_u32(bars.w_full), we0 = smem_u32(bars.w_empty);
    const uint32_t wgf = smem_u32(&bars.wg_full), wge = smem_u32(&bars.wg_empty);

    if (warp == 4) {
        // ------------------------------------------------------------ loader
        if (lane == 0) {
            uint32_t n = 0, wcount = 0;
            int cur = -1;
            const uint64_t pol = l2_evict_first_policy();
            for (long long i = i0; i < i1; ++i, ++n) {
                const int blk = (int)(i / p.ntiles), tile = p.reverse ? p.ntiles - 1 - (int)(i % p.ntiles) : (int)(i % p.ntiles);
                if (blk != cur) {
                    const uint32_t wp = wcount & 1;
                    if (!mbar_wait(we0 + wp * 8, ((wcount >> 1) & 1) ^ 1, p.status, dead, kErrSlotWait)) break;
                    mbar_expect_tx(wf0 + wp * 8, kOpBytes);
                    tma_load_2d(w0 + wp * kOpBytes, &tm_w, 0, blk * kB, wf0 + wp * 8);
                    tma_load_2d(w0 + wp * kOpBytes + kHalfBytes, &tm_w, 64, blk * kB, wf0 + wp * 8);
                    if (wcount == 0) pdl_wait();
                    ++wcount;
                    cur = blk;
                }
                const uint32_t s = n % SLOTS;
                if (!mbar_wait(empty0 + s * 8, ((n / SLOTS) & 1) ^ 1, p.status, dead, kErrSlotWait)) break;
                mbar_expect_tx(full0 + s * 8, kSlotBytes);
                load_operand_last_use<T0_LD>(ring0 + s * kSlotBytes, &tm_t0, p.t0_base, blk, tile, full0 + s * 8, pol);
                if (WG) load_operand_last_use<T1_LD>(ring0 + s * kSlotBytes + kOpBytes, &tm_t1, p.t1_base, blk, tile, full0 + s * 8, pol);
            }
        }
    } else if (warp == 6) {
        // ------------------------------------------------------------ the consumed slab of the intermediate leaves L2
        if (T0_LD == kLdC) {
            uint32_t n = 0;
            for (long long i = i0; i < i1; ++i, ++n) {
                const int blk = (int)(i / p.ntiles), tile = p.reverse ? p.ntiles - 1 - (int)(i % p.ntiles) : (int)(i % p.ntiles);
                const uint32_t s = n % SLOTS;
                if (!mbar_wait(full0 + s * 8, (n / SLOTS) & 1, p.status, dead, kErrTmaWait)) break;
                if (p.discard_t0) discard_slab(p.t0_base + ((size_t)tile * kB + blk) * kOpBytes, lane);
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + s * 8);
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_main = W_IS_A ? make_idesc_bf16(128, 128, W_MN, T0_MN) : make_idesc_bf16(128, 128, T0_MN, W_MN);
            constexpr uint32_t idesc_wg = make_idesc_bf16(128, 128, 0, T1_MN);
            uint32_t n = 0, wcount = 0, wp = 0;
            int cur = -1;
            bool wg_first = true;
            for (long long i = i0; i < i1; ++i, ++n) {
                const int blk = (int)(i / p.ntiles);
                if (blk != cur) {
                    wp = wcount & 1;
                    if (!mbar_wait(wf0 + wp * 8, (wcount >> 1) & 1, p.status, dead, kErrTmaWait)) break;
                    if (WG) {
                        // the previous block's sums have left TMEM
                        if (!mbar_wait(wge, (wcount & 1) ^ 1, p.status, dead, kErrTmemWait)) break;
                        wg_first = true;
                    }
                    ++wcount;
                    cur = blk;
                }
                const uint32_t buf = n & 1, s = n % SLOTS;
                if (MAIN) {
                    if (!mbar_wait(acce0 + buf * 8, ((n >> 1) & 1) ^ 1, p.status, dead, kErrTmemWait)) break;
                }
                if (!mbar_wait(full0 + s * 8, (n / SLOTS) & 1, p.status, dead, kErrTmaWait)) break;
                tc_fence_after();
                const uint32_t t0 = ring0 + s * kSlotBytes, t1 = t0 + kOpBytes, w = w0 + wp * kOpBytes;
                if (MAIN) {
                    const uint32_t d = tmem_base + buf * 128;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t dw = op_desc(w, W_MN, ks), dt = op_desc(t0, T0_MN, ks);
                        mma_f16_ss(d, W_IS_A ? dw : dt, W_IS_A ? dt : dw, idesc_main, ks != 0);
                    }
                    mma_commit(accf0 + buf * 8);
                }
                if (WG) {
                    const uint32_t d = tmem_base + 256;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        mma_f16_ss(d, op_desc(t0, false, ks), op_desc(t1, T1_MN, ks), idesc_wg, !(wg_first && ks == 0));
                    wg_first = false;
                }
                mma_commit(empty0 + s * 8);
                if (i + 1 == i1 || (int)((i + 1) / p.ntiles) != blk) {
                    mma_commit(we0 + wp * 8);
                    if (WG) mma_commit(wgf);
                }
            }
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------ epilogue (warps 0-3 = TMEM lanes 32w..32w+31)
        const int row = warp * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
        uint32_t n = 0, nchunk = 0, nb = 0;
        bool ok = true;
        for (long long i = i0; ok && i < i1; ++i, ++n) {
            const int blk = (int)(i / p.ntiles), tile = p.reverse ? p.ntiles - 1 - (int)(i % p.ntiles) : (int)(i % p.ntiles);
            const int xorp = ST == kStP ? (blk & 7) : 0;
            if (MAIN) {
                const uint32_t buf = n & 1;
                if (!mbar_wait(accf0 + buf * 8, (n >> 1) & 1, p.status, dead, kErrMmaWait)) break;
                tc_fence_after();
#pragma unroll 1
                for (int h = 0; h < 2; ++h, ++nchunk) {
                    const uint32_t stg = staging0 + (nchunk & 1) * kHalfBytes;
                    // this staging tile is free once the store issued two chunks ago has read it
                    if (threadIdx.x == 0) tma_store_wait_read<1>();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    uint32_t v[4][16];
#pragma unroll
                    for (int q = 0; q < 4; ++q) tmem_ld16(lane_base + buf * 128 + h * 64 + q * 16, v[q]);
                    tmem_ld_wait();
                    if (h == 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(acce0 + buf * 8);
                    }
                    const uint32_t dst = stg + row * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint32_t *w = &v[c >> 1][(c & 1) * 8];
                        const uint32_t o0 = pack_bf16(__uint_as_float(w[0]), __uint_as_float(w[1]));
                        const uint32_t o1 = pack_bf16(__uint_as_float(w[2]), __uint_as_float(w[3]));
                        const uint32_t o2 = pack_bf16(__uint_as_float(w[4]), __uint_as_float(w[5]));
                        const uint32_t o3 = pack_bf16(__uint_as_float(w[6]), __uint_as_float(w[7]));
                        // producer pieces: the store un-swizzles by the row, the slab wants the chunks XORed with blk % 8
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + ((c ^ xorp ^ (row & 7)) << 4)),
                                     "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                    }
                    fence_proxy_async_smem();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (threadIdx.x == 0) {
                        // a token-major output is final (written once, not read by this chain): evict-first
                        if (ST == kStX) tma_store_2d_stream(&tm_out, stg, blk * kB + h * 64, tile * 128, l2_evict_first_policy());
                        else tma_store_5d_keep(&tm_out, stg, 0, blk, h, 0, tile, l2_evict_last_policy());
                        tma_store_commit();
                    }
                }
            }
            if (WG && (i + 1 == i1 || (int)((i + 1) / p.ntiles) != blk)) {
                // the block's token sums are complete: store them to dW[blk] or add them to it (one writer per element).
                // They leave like the main product's tiles: 32 columns at a time through the swizzled staging tiles and a
                // tiled TMA store / reduce-add (plain 16-byte stores from 128 threads, each to its own row, cost 2.7 us here)
                if (!mbar_wait(wgf, nb & 1, p.status, dead, kErrMmaWait)) break;
                tc_fence_after();
#pragma unroll 1
                for (int q = 0; q < 4; ++q, ++nchunk) {
                    const uint32_t stg = staging0 + (nchunk & 1) * kHalfBytes;
                    if (threadIdx.x == 0) tma_store_wait_read<1>();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    uint32_t v[2][16];
                    tmem_ld16(lane_base + 256 + q * 32, v[0]);
                    tmem_ld16(lane_base + 256 + q * 32 + 16, v[1]);
                    tmem_ld_wait();
                    const uint32_t dst = stg + row * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint32_t *w = &v[c >> 2][(c & 3) * 4];
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + ((c ^ (row & 7)) << 4)), "r"(w[0]),
                                     "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
                    }
                    fence_proxy_async_smem();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (threadIdx.x == 0) {
                        if (p.overwrite) tma_store_2d_plain(&tm_dw, stg, q * 32, blk * kB);
                        else tma_reduce_add_2d(&tm_dw, stg, q * 32, blk * kB);
                        tma_store_commit();
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(wge);
                ++nb;
            }
        }
        if ((MAIN || WG) && threadIdx.x == 0) tma_store_wait_all<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

// ---------------------------------------------------------------------------------------------------------
// 128 x 128 plane transposes between a token-major tensor v[t][pl*128 + r] and an intermediate:
// TO_PLANES = false: consumer slab pl (rows r, tokens along the row) -> token-major (the outer P of step 3 of the
// forward pass); true: token-major -> producer pieces of plane pl (row r of the transposed tile goes to consumer r;
// first step of the adjoint).  In and out are each two halves of [128 rows][64 columns] with the 128-byte swizzle;
// four warps move 8 x 8 tiles with ldmatrix.trans / stmatrix (conflict-free under the swizzle).
constexpr int kTrIn = 3, kTrOut = 2;
constexpr int kTrThreads = 5 * 32;
constexpr int kTrSmem = (kTrIn + kTrOut) * kOpBytes + 1024;

struct TransposeParams {
    unsigned *status;
    const char *in_base;                 // the intermediate (TO_PLANES = false)
    int ntiles, nplanes;                 // planes per tile (128)
    long long skip_item;                 // injected fault (tests only), else -1
};

template <bool TO_PLANES>
__global__ void __launch_bounds__(kTrThreads, 1)
plane_transpose_kernel(const __grid_constant__ CUtensorMap tm_in, const __grid_constant__ CUtensorMap tm_out,
                       const TransposeParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full[kTrIn], empty[kTrIn];
    __shared__ int dead_s;
    const uint32_t in0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t out0 = in0 + kTrIn * kOpBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *dead = &dead_s;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kTrIn; ++s) {
            mbar_init(smem_u32(&full[s]), 1);
            mbar_init(smem_u32(&empty[s]), 4);
        }
        fence_mbar_init();
        dead_s = 0;
        tma_prefetch_desc(&tm_in); tma_prefetch_desc(&tm_out);
    }
    pdl_launch_dependents();
    __syncthreads();
    pdl_wait();
    // items (tile, plane), tile-major, dealt out round robin: the whole grid moves through the tiles together, so the
    // next launch of the chain can start with the tiles written last (still in L2)
    const long long total = (long long)p.ntiles * p.nplanes;
    const long long i0 = blockIdx.x, istep = gridDim.x;

    if (warp == 4) {
        if (lane == 0) {
            uint32_t n = 0;
            const uint64_t pol = l2_evict_first_policy();
            int last_fill[kTrIn];
#pragma unroll
            for (int s = 0; s < kTrIn; ++s) last_fill[s] = -1;
            for (long long i = i0; i < total; i += istep, ++n) {
                const int tile = (int)(i / p.nplanes), pl = (int)(i % p.nplanes);
                const uint32_t s = n % kTrIn;
                if (!mbar_wait(smem_u32(&empty[s]), ((n / kTrIn) & 1) ^ 1, p.status, dead, kErrSlotWait)) break;
                if (i == p.skip_item) continue;
                mbar_expect_tx(smem_u32(&full[s]), kOpBytes);
                load_operand_last_use<TO_PLANES ? kLdX : kLdC>(in0 + s * kOpBytes, &tm_in, p.in_base, pl, tile, smem_u32(&full[s]), pol);
                last_fill[s] = (int)(n / kTrIn);
            }
            if (*dead) {
                // unwinding after a wait that ran out: no copy into this CTA's shared memory may outlive the CTA
#pragma unroll
                for (int s = 0; s < kTrIn; ++s)
                    if (last_fill[s] >= 0)
                        for (int spin = 0; spin < (1 << 22) && !mbar_try_wait(smem_u32(&full[s]), last_fill[s] & 1); ++spin) { }
            }
        }
    } else {
        uint32_t n = 0;
        for (long long i = i0; i < total; i += istep, ++n) {
            const int tile = (int)(i / p.nplanes), pl = (int)(i % p.nplanes);
            const uint32_t s = n % kTrIn, ob = out0 + (n & 1) * kOpBytes, ib = in0 + s * kOpBytes;
            // the output buffer used two items ago has been read by its stores
            if (threadIdx.x == 0) tma_store_wait_read<1>();
            if (!mbar_wait(smem_u32(&full[s]), (n / kTrIn) & 1, p.status, dead, kErrTmaWait)) break;
            asm volatile("bar.sync 1, 128;" ::: "memory");
            // in[r][c] -> out[c][r]; warp w takes source rows 32w..32w+31 (four row octets), all 16 column octets
#pragma unroll 1
            for (int ro = 0; ro < 4; ++ro) {
                const int r0 = warp * 32 + ro * 8;
#pragma unroll
                for (int cq = 0; cq < 4; ++cq) {
                    // four 8 x 8 tiles: source rows r0..r0+7, column octets 4cq..4cq+3
                    const int mi = lane >> 3, ri = lane & 7;
                    const int co = cq * 4 + mi;                                  // column octet 0..15
                    const int sr = r0 + ri;
                    const uint32_t src = ib + (co >> 3) * kHalfBytes + sr * 128 + (((co & 7) ^ (sr & 7)) << 4);
                    uint32_t a, b, c, d;
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(src) : "memory");
                    // destination tile of matrix mi: rows co*8..co*8+7 (source columns), column octet r0/8
                    // producer pieces: the store un-swizzles by the row, the slab wants the chunks XORed with pl % 8
                    const int dr = co * 8 + ri, dco = (r0 >> 3) ^ (TO_PLANES ? (pl & 7) : 0);
                    const uint32_t dst = ob + (r0 >> 6) * kHalfBytes + dr * 128 + (((dco & 7) ^ (dr & 7)) << 4);
                    asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(a),
                                 "r"(b), "r"(c), "r"(d) : "memory");
                }
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&empty[s]));
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (threadIdx.x == 0) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (TO_PLANES) tma_store_5d_keep(&tm_out, ob + h * kHalfBytes, 0, pl, h, 0, tile, l2_evict_last_policy());
                    else tma_store_2d(&tm_out, ob + h * kHalfBytes, pl * kB + h * 64, tile * 128);
                }
                tma_store_commit();
            }
        }
        if (threadIdx.x == 0) tma_store_wait_all<0>();
    }
}

// ---------------------------------------------------------------------------------------------------------
// The whole forward pass in one persistent launch: CTA b (one per SM, 128 of them) owns block b of every step and
// walks the token tiles; at step s it runs
//     A: D_b[j][t] = R_b x_b(tile s)            -> pieces of u'[tile s] (row j to consumer j)      (stage 1)
//     B: D_b[l][t] = L_b u'_b(tile s - LAG)     -> pieces of w'[(tile s - LAG) % RING]             (stage 2)
//     C: y[t][b*128 + j] = slab b of w'[tile s - 2 LAG], transposed                                (outer P)
// u' and w' have the layout of the three-launch chain (a producer writes 128-byte pieces 32 KB apart, a consumer
// reads its 32 KB slab with one linear bulk copy).  An SM can push about 28.6 bytes per clock towards L2 whatever
// the mechanism (load/store units or bulk copies; measured), i.e. the 96 KB a CTA writes per step cost 3.4 k
// cycles: the stores, not the loads (70 B/clk) or the tensor pipe, bound this kernel.  Rows leave through the
// load/store units from dedicated store warps (8 lanes per 128-byte piece); publishing a slab costs a memory fence
// of a few thousand cycles, so kStoreSets warp pairs take the items in turn.  TMA stores were tried instead (tiled:
// the TMA unit then carries 160 KB per step at its 30 B/clk for tiled copies; linear bulk copies of contiguous
// slabs with the consumers gathering rows by 16-byte asynchronous copies: no faster, the store thread waits on the
// same 28.6 B/clk) and are not kept.
// B needs the rows that all 128 CTAs wrote in A LAG steps earlier, C those of B: one counter per tile and stage,
// bumped by each CTA's store warps when their rows are in memory and polled (bounded) by the consumer's loader.  Dependencies only point to earlier steps, every CTA is resident (the launch is refused otherwise), so
// the waits cannot deadlock; the lag hides them.  x is read once and y written once (by the load/store units,
// straight from the transposed plane); u' is also kept for the backward call, w' lives in a ring of RING tiles
// that stays in L2.
#ifndef MONARCH_FUSED_LAG
#define MONARCH_FUSED_LAG 3
#endif
constexpr int kFusedLag = MONARCH_FUSED_LAG, kFusedRing = 2 * kFusedLag + 2;
constexpr int kStoreSets = 3;                // store-warp pairs taking the items in turn
constexpr int kFusedThreads = (13 + 2 * kStoreSets) * 32;   // warps 0-3 epilogue, 4-7 transposers, 8 u' loader, 9 MMA, 10.. store warps, then plane loader, L2 prefetch, x loader
constexpr int kFusedPrefetch = 2;           // steps between the L2 prefetch of an x tile and its load
constexpr int kFusedSmem = 2 * kOpBytes /* R_b, L_b */ + 2 * kOpBytes /* operand ring */ + kStagingBytes +
                           2 * kOpBytes /* plane in, out */ + 1024;
constexpr unsigned kFusedCounters = 8192;    // tiles per counter array (two arrays in the 64 KB after the status word)

struct FusedParams {
    unsigned *status;
    unsigned *cnt1, *cnt2;                   // per tile: store warps (two per CTA) whose stage-1 / stage-2 rows are in memory
    char *u, *w, *y;                         // u' planes, w' ring, output
    const char *x;                           // input, for the L2 prefetch hints only (the data path goes through TMA)
    long long tokens;
    int ntiles;
    long long *trace;                        // debug builds: per-CTA cycle sums of the waits, else null
};

#ifdef MONARCH_TRACE
#define FT0() const long long ft0_ = clock64()
#define FACC(v) v += clock64() - ft0_
#define FOUT(site, v) do { if (p.trace) p.trace[blockIdx.x * 16 + (site)] = (v); } while (0)
#else
#define FT0() do { } while (0)
#define FACC(v) do { } while (0)
#define FOUT(site, v) do { } while (0)
#endif

struct FusedBars {
    uint64_t w_full;
    uint64_t full[2], empty[2];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t st_full[2 * kStoreSets], st_free[2];   // st_full: one per store-warp set and staging half
    uint64_t tr_full, tr_empty;
};

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void fence_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

// Wait (bounded) until all `need` producers of a tile have published; the last of the `consumers` to get here puts
// the counter back to zero for the next call.
__device__ __forceinline__ bool wait_counter(unsigned *ctr, unsigned need, unsigned consumers, unsigned *status,
                                             volatile int *dead)
{
    if (ld_acquire_gpu(ctr) < need) {
        const unsigned long long t0 = global_timer_ns(), limit = wait_limit_ns(status);
        while (ld_acquire_gpu(ctr) < need) {
            if (*dead || global_timer_ns() - t0 > limit) {
                *dead = 1;
                atomicCAS(status, 0u, (unsigned)kErrPeerWait);
                return false;
            }
            __nanosleep(64);                     // 128 CTAs poll this word; a hot loop only costs power
        }
    }
    if (atomicAdd(ctr, 1u) + 1 == need + consumers) atomicExch(ctr, 0u);
    fence_async_global();
    return true;
}

__global__ void __launch_bounds__(kFusedThreads, 1)
chain_fused_fwd_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_R,
                       const __grid_constant__ CUtensorMap tm_L, const FusedParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) FusedBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead_s;
    __shared__ int x_prog_s;                 // x tiles the loader has asked for

    const uint32_t w0 = (smem_u32(smem_raw) + 1023u) & ~1023u;          // R_b, L_b
    const uint32_t ring0 = w0 + 2 * kOpBytes;
    const uint32_t staging0 = ring0 + 2 * kOpBytes;
    const uint32_t trin = staging0 + kStagingBytes, trout = trin + kOpBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = (int)blockIdx.x;
    volatile int *dead = &dead_s;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars.w_full), 1);
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&bars.full[a]), 1);
            mbar_init(smem_u32(&bars.empty[a]), 1);
            mbar_init(smem_u32(&bars.acc_full[a]), 1);
            mbar_init(smem_u32(&bars.acc_empty[a]), 4);
            for (int k = 0; k < kStoreSets; ++k) mbar_init(smem_u32(&bars.st_full[k * 2 + a]), 4);
            mbar_init(smem_u32(&bars.st_free[a]), 1);
        }
        mbar_init(smem_u32(&bars.tr_full), 1);
        mbar_init(smem_u32(&bars.tr_empty), 4);
        fence_mbar_init();
        dead_s = 0;
        x_prog_s = 0;
        tma_prefetch_desc(&tm_x); tma_prefetch_desc(&tm_R); tma_prefetch_desc(&tm_L);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 256);
        tmem_relinquish();
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    if (!(warp == 8 && lane == 0)) pdl_wait();          // the loader waits after it has asked for the weights

    const int nt = p.ntiles, nsteps = nt + 2 * kFusedLag;
    const uint32_t full0 = smem_u32(bars.full), empty0 = smem_u32(bars.empty);
    const uint32_t accf0 = smem_u32(bars.acc_full), acce0 = smem_u32(bars.acc_empty);
    const uint32_t stf0 = smem_u32(bars.st_full), stfree0 = smem_u32(bars.st_free);
    const uint32_t trf = smem_u32(&bars.tr_full), tre = smem_u32(&bars.tr_empty);

    if (warp == 8) {
        // ------------------------------------------------------------ loader
        if (lane == 0) {
            const uint32_t wbar = smem_u32(&bars.w_full);
            mbar_expect_tx(wbar, 2 * kOpBytes);
            tma_load_2d(w0, &tm_R, 0, b * kB, wbar);
            tma_load_2d(w0 + kHalfBytes, &tm_R, 64, b * kB, wbar);
            tma_load_2d(w0 + kOpBytes, &tm_L, 0, b * kB, wbar);
            tma_load_2d(w0 + kOpBytes + kHalfBytes, &tm_L, 64, b * kB, wbar);
            pdl_wait();
            // the u' slabs of stage 2 go through ring slot 1; the x tiles have their own loader and slot 0, so that a wait
            // for the other CTAs here never holds back this CTA's own stage 1 (whose rows the others are waiting for)
            [[maybe_unused]] long long wc = 0, wb = 0;
            const uint64_t pol = l2_evict_first_policy();
            for (int tb = 0; tb < nt; ++tb) {
                { FT0(); if (!wait_counter(p.cnt1 + tb, 2 * kB, kB, p.status, dead)) break; FACC(wc); }
                { FT0(); if (!mbar_wait(empty0 + 8, (tb & 1) ^ 1, p.status, dead, kErrSlotWait)) break; FACC(wb); }
                mbar_expect_tx(full0 + 8, kOpBytes);
                bulk_load_linear_last_use(ring0 + kOpBytes, p.u + ((size_t)tb * kB + b) * kOpBytes, kOpBytes, full0 + 8, pol);
            }
            FOUT(1, wc); FOUT(2, wb);
        }
    } else if (warp == 12 + 2 * kStoreSets) {
        // ------------------------------------------------------------ x loader (ring slot 0)
        if (lane == 0) {
            pdl_wait();
            const uint64_t pol = l2_evict_first_policy();
            [[maybe_unused]] long long wa = 0;
            for (int s = 0; s < nt; ++s) {
                { FT0(); if (!mbar_wait(empty0, (s & 1) ^ 1, p.status, dead, kErrSlotWait)) break; FACC(wa); }
                mbar_expect_tx(full0, kOpBytes);
                tma_load_2d_last_use(ring0, &tm_x, b * kB, s * 128, full0, pol);
                tma_load_2d_last_use(ring0 + kHalfBytes, &tm_x, b * kB + 64, s * 128, full0, pol);
                *reinterpret_cast<volatile int *>(&x_prog_s) = s + 1;
            }
            FOUT(0, wa);
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && mbar_wait(smem_u32(&bars.w_full), 0, p.status, dead, kErrTmaWait)) {
            constexpr uint32_t idesc_a = make_idesc_bf16(128, 128, 0, 0), idesc_b = make_idesc_bf16(128, 128, 0, 1);
            uint32_t g = 0;
            bool ok = true;
            [[maybe_unused]] long long wa = 0, wf = 0;
            for (int s = 0; ok && s < nsteps; ++s) {
#pragma unroll
                for (int ki = 0; ki < 2; ++ki) {
                    const int kind = 1 - ki;                      // stage 2 of the older tile first, then stage 1
                    const int tile = kind == 0 ? s : s - kFusedLag;
                    if (tile < 0 || tile >= nt) continue;
                    // accumulators alternate item by item; the operand comes from the slot of its kind (slot use = tile)
                    const uint32_t buf = g & 1, sl = kind;
                    { FT0(); if (!mbar_wait(acce0 + buf * 8, ((g >> 1) & 1) ^ 1, p.status, dead, kErrTmemWait)) { ok = false; break; } FACC(wa); }
                    { FT0(); if (!mbar_wait(full0 + sl * 8, tile & 1, p.status, dead, kErrTmaWait)) { ok = false; break; } FACC(wf); }
                    tc_fence_after();
                    const uint32_t t0 = ring0 + sl * kOpBytes, w = w0 + kind * kOpBytes, d = tmem_base + buf * 128;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        mma_f16_ss(d, op_desc(w, false, ks), op_desc(t0, kind == 1, ks), kind == 0 ? idesc_a : idesc_b, ks != 0);
                    mma_commit(empty0 + sl * 8);
                    mma_commit(accf0 + buf * 8);
                    ++g;
                }
            }
            FOUT(3, wa); FOUT(4, wf);
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------ epilogue: TMEM -> bf16 -> staging halves
        const int row = warp * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
        uint32_t g = 0;
        bool ok = true;
        [[maybe_unused]] long long wa = 0, ws = 0;
        [[maybe_unused]] const long long te0 = clock64();
        for (int s = 0; ok && s < nsteps; ++s) {
#pragma unroll 1
            for (int ki = 0; ki < 2; ++ki) {
                const int kind = 1 - ki;
                const int tile = kind == 0 ? s : s - kFusedLag;
                if (tile < 0 || tile >= nt) continue;
                const uint32_t buf = g & 1;
                { FT0(); if (!mbar_wait(accf0 + buf * 8, (g >> 1) & 1, p.status, dead, kErrMmaWait)) { ok = false; break; } FACC(wa); }
                tc_fence_after();
#pragma unroll 1
                for (int h = 0; h < 2; ++h) {
                    uint32_t v[4][16];
#pragma unroll
                    for (int q = 0; q < 4; ++q) tmem_ld16(lane_base + buf * 128 + h * 64 + q * 16, v[q]);
                    tmem_ld_wait();
                    if (h == 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(acce0 + buf * 8);
                    }
                    // staging half h is free once the store of the previous item's half h has read it
                    { FT0(); if (!mbar_wait(stfree0 + h * 8, (g & 1) ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; } FACC(ws); }
                    const uint32_t dst = staging0 + h * kHalfBytes + row * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint32_t *w = &v[c >> 1][(c & 1) * 8];
                        const uint32_t o0 = pack_bf16(__uint_as_float(w[0]), __uint_as_float(w[1]));
                        const uint32_t o1 = pack_bf16(__uint_as_float(w[2]), __uint_as_float(w[3]));
                        const uint32_t o2 = pack_bf16(__uint_as_float(w[4]), __uint_as_float(w[5]));
                        const uint32_t o3 = pack_bf16(__uint_as_float(w[6]), __uint_as_float(w[7]));
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + ((c ^ (row & 7)) << 4)),
                                     "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(stf0 + ((g % kStoreSets) * 2 + h) * 8);
                }
                if (!ok) break;
                ++g;
            }
        }
        if (threadIdx.x == 0) { FOUT(5, wa); FOUT(6, ws); FOUT(7, clock64() - te0); }
    } else if (warp >= 10 && warp < 10 + 2 * kStoreSets) {
        // ------------------------------------------------------------ store warps (per set: one per staging half):
        // rows of D leave as 128-byte pieces through the load/store units (8 lanes per row), then this warp's part
        // of the tile is published
        const int h = (warp - 10) & 1, set = (warp - 10) >> 1;
        const uint32_t src = staging0 + h * kHalfBytes;
        uint32_t g = 0;
        bool ok = true;
        [[maybe_unused]] long long wf = 0;
        [[maybe_unused]] const long long ts0 = clock64();
        for (int s = 0; ok && s < nsteps; ++s) {
#pragma unroll 1
            for (int ki = 0; ki < 2; ++ki) {
                const int kind = 1 - ki;
                const int tile = kind == 0 ? s : s - kFusedLag;
                if (tile < 0 || tile >= nt) continue;
                if ((int)(g % kStoreSets) != set) { ++g; continue; }
                { FT0(); if (!mbar_wait(stf0 + (set * 2 + h) * 8, (g / kStoreSets) & 1, p.status, dead, kErrMmaWait)) { ok = false; break; } FACC(wf); }
                // row r of D is the piece [tile][c = r][h][p = b] of the intermediate, chunks XORed with b % 8
                char *dst = (kind == 0 ? p.u + (size_t)tile * (kB * kOpBytes) : p.w + (size_t)(tile % kFusedRing) * (kB * kOpBytes)) +
                            h * kHalfBytes + b * 128 + (((lane & 7) ^ (b & 7)) << 4);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 v[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int r = (q * 8 + i) * 4 + (lane >> 3);
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v[i].x), "=r"(v[i].y), "=r"(v[i].z), "=r"(v[i].w)
                                     : "r"(src + r * 128 + (((lane & 7) ^ (r & 7)) << 4)) : "memory");
                    }
                    if (q == 3) {
                        // the staging half is in registers: hand it back to the epilogue
                        __syncwarp();
                        if (lane == 0) mbar_arrive(stfree0 + h * 8);
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int r = (q * 8 + i) * 4 + (lane >> 3);
                        *reinterpret_cast<uint4 *>(dst + (size_t)r * kOpBytes) = v[i];
                    }
                }
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd((kind == 0 ? p.cnt1 : p.cnt2) + tile, 1u);
                ++g;
            }
        }
        if (warp == 10 && lane == 0) { FOUT(8, wf); FOUT(9, clock64() - ts0); }
    } else if (warp == 11 + 2 * kStoreSets) {
        // ------------------------------------------------------------ L2 prefetch of x: the operand ring has two slots, so
        // an x tile is asked for only when the MMAs two items back are done - one DRAM latency too late.  This warp asks
        // L2 for the tile kFusedPrefetch steps ahead (256-byte rows, one token apart) through the load/store units.
        volatile int *x_prog = &x_prog_s;
        const unsigned long long limit = wait_limit_ns(p.status);
        for (int s = 0; s < nt; ++s) {
            if (s >= *x_prog + kFusedPrefetch) {
                const unsigned long long t0 = global_timer_ns();
                while (s >= *x_prog + kFusedPrefetch && !*dead && global_timer_ns() - t0 < limit) __nanosleep(256);
                if (s >= *x_prog + kFusedPrefetch) break;
            }
            const char *a = p.x + ((size_t)s * 128 + (lane >> 1)) * ((size_t)kB * kB * 2) + b * 256 + (lane & 1) * 128;
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if ((long long)s * 128 + i * 16 + (lane >> 1) < p.tokens)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(a + (size_t)i * 16 * ((size_t)kB * kB * 2)));
        }
    } else if (warp == 10 + 2 * kStoreSets) {
        // ------------------------------------------------------------ plane loader
        if (lane == 0) {
            uint32_t c = 0;
            [[maybe_unused]] long long wc = 0, we = 0;
            const uint64_t pol = l2_evict_first_policy();
            for (int s = 2 * kFusedLag; s < nsteps; ++s, ++c) {
                const int tc = s - 2 * kFusedLag;
                { FT0(); if (!wait_counter(p.cnt2 + tc, 2 * kB, kB, p.status, dead)) break; FACC(wc); }
                { FT0(); if (!mbar_wait(tre, (c & 1) ^ 1, p.status, dead, kErrSlotWait)) break; FACC(we); }
                mbar_expect_tx(trf, kOpBytes);
                bulk_load_linear_last_use(trin, p.w + ((size_t)(tc % kFusedRing) * kB + b) * kOpBytes, kOpBytes, trf, pol);
            }
            FOUT(10, wc); FOUT(11, we);
        }
    } else {
        // ------------------------------------------------------------ transposers (warps 4-7): plane b of w' -> y
        const int tw = warp - 4;
        uint32_t c = 0;
        [[maybe_unused]] long long wf = 0;
        [[maybe_unused]] const long long tt0 = clock64();
        for (int s = 2 * kFusedLag; s < nsteps; ++s, ++c) {
            const int tile = s - 2 * kFusedLag;
            { FT0(); if (!mbar_wait(trf, c & 1, p.status, dead, kErrTmaWait)) break; FACC(wf); }
            // every warp has copied its rows of the previous plane out of the output buffer
            asm volatile("bar.sync 2, 128;" ::: "memory");
#pragma unroll 1
            for (int ro = 0; ro < 4; ++ro) {
                const int r0 = tw * 32 + ro * 8;
#pragma unroll
                for (int cq = 0; cq < 4; ++cq) {
                    const int mi = lane >> 3, ri = lane & 7;
                    const int co = cq * 4 + mi, sr = r0 + ri;
                    const uint32_t src = trin + (co >> 3) * kHalfBytes + sr * 128 + (((co & 7) ^ (sr & 7)) << 4);
                    uint32_t a, bq, cc, d;
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(a), "=r"(bq), "=r"(cc), "=r"(d) : "r"(src) : "memory");
                    const int dr = co * 8 + ri, dco = r0 >> 3;
                    const uint32_t dst = trout + (dco >> 3) * kHalfBytes + dr * 128 + (((dco & 7) ^ (dr & 7)) << 4);
                    asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(a),
                                 "r"(bq), "r"(cc), "r"(d) : "memory");
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(tre);
            asm volatile("bar.sync 2, 128;" ::: "memory");
            // rows t = 32 tw .. 32 tw + 31 of y[t][b*128 ..], two 128-byte pieces each; rows past the last token stay put
            char *yrow = p.y + ((size_t)tile * 128) * kOpBytes + b * 256 + (lane & 7) * 16;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint4 v[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = tw * 32 + i * 4 + (lane >> 3);
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v[i].x), "=r"(v[i].y), "=r"(v[i].z), "=r"(v[i].w)
                                 : "r"(trout + hh * kHalfBytes + r * 128 + (((lane & 7) ^ (r & 7)) << 4)) : "memory");
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int t = tw * 32 + i * 4 + (lane >> 3);
                    if ((long long)tile * 128 + t < p.tokens)
                        asm volatile("st.global.cs.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(yrow + (size_t)t * kOpBytes + hh * 128),
                                     "r"(v[i].x), "r"(v[i].y), "r"(v[i].z), "r"(v[i].w) : "memory");
                }
            }
        }
        if (warp == 4 && lane == 0) { FOUT(12, wf); FOUT(13, clock64() - tt0); }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 256);
}

// ---------------------------------------------------------------------------------------------------------
struct Maps {
    CUtensorMap x2d;       // token-major [tokens][n], box 128 rows x 64 columns
    CUtensorMap p4d;       // planes [tile][p][q][t], box = rows q of one p
    CUtensorMap q4d;       // planes, box = rows p of one q
};

int map_tokens(CUtensorMap *m, const void *v, int64_t tokens)
{
    return encode_tmap_2d(m, v, (uint64_t)tokens, (uint64_t)kB * kB, (uint64_t)kB * kB * 2, 128, 64, 128);
}
int map_weights(CUtensorMap *m, const void *W)
{
    return encode_tmap_2d(m, W, (uint64_t)kB * kB, kB, kB * 2, 128, 64, 128);
}
// producer pieces of an intermediate [tile][c][h][p][64 t]: box = the 128-byte pieces of one producer and half, all c
int map_pieces(CUtensorMap *m, const void *v, int ntiles)
{
    const uint64_t dims[5] = {64, 128, 2, 128, (uint64_t)ntiles}, strides[4] = {128, 16384, 32768, 4194304};
    const uint32_t box[5] = {64, 1, 1, 128, 1};
    return encode_tmap_nd(m, v, 2, 5, dims, strides, box, 128);
}

int device_sms(int *sms) { return current_device_sms(sms); }

// Launch with programmatic stream serialization: the kernel may start while its predecessor in the stream drains.
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kern)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t s, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// t0 / t1: a tensor map (token-major tensor) or the base pointer of an intermediate, whichever the load kind reads
struct Src {
    const CUtensorMap *map;
    const char *base;
};

template <int T0_LD, bool W_IS_A, bool W_MN, bool T0_MN, int ST, bool WG, int T1_LD, bool T1_MN, bool MAIN>
int launch_gemm(Src t0, Src t1, const CUtensorMap &w, const CUtensorMap &out, float *dW, int ntiles, unsigned *status, cudaStream_t s,
                int overwrite = 0, int reverse = 0, int discard_t0 = 0)
{
    constexpr int SLOTS = WG ? 2 : 3;
    constexpr int smem = 2 * kOpBytes + SLOTS * (WG ? 2 : 1) * kOpBytes + kStagingBytes + 1024;
    auto kern = chain_gemm_kernel<T0_LD, W_IS_A, W_MN, T0_MN, ST, WG, T1_LD, T1_MN, MAIN, SLOTS>;
    int sms = 0;
    MONARCH_TRY(device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    ChainParams p;
    p.status = status;
    p.dW = dW;
    p.overwrite = overwrite;
    p.reverse = reverse;
    p.discard_t0 = discard_t0;
    p.t0_base = t0.base;
    p.t1_base = t1.base;
    p.ntiles = ntiles;
    p.nblk = kB;
    long long grid = WG ? kB : (long long)kB * ntiles;
    if (grid > sms) grid = sms;
    // the weight gradient [block * 128 + row][128] fp32 in pieces of 32 columns x 128 rows (128-byte rows, swizzled)
    CUtensorMap mdw = w;
    if (WG) {
        const uint64_t dims[2] = {(uint64_t)kB, (uint64_t)kB * kB}, strides[1] = {(uint64_t)kB * sizeof(float)};
        const uint32_t box[2] = {32, 128};
        MONARCH_TRY(encode_tmap_nd(&mdw, dW, 4, 2, dims, strides, box, 128));
    }
    // a load kind that reads a base pointer ignores its map: pass any valid one
    MONARCH_CUDA_TRY(launch_chained(kern, (unsigned)grid, kThreads, smem, s, t0.map ? *t0.map : w, t1.map ? *t1.map : w, w, out, mdw, p));
    note_launch();
    return MONARCH_OK;
}

template <bool TO_PLANES>
int launch_transpose(Src in, const CUtensorMap &out, int ntiles, unsigned *status, cudaStream_t s)
{
    int sms = 0;
    MONARCH_TRY(device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(plane_transpose_kernel<TO_PLANES>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTrSmem));
    TransposeParams p;
    p.status = status;
    p.in_base = in.base;
    p.ntiles = ntiles;
    p.nplanes = kB;
    p.skip_item = g_skip_load.exchange(-1);
    long long grid = (long long)ntiles * kB;
    if (grid > sms) grid = sms;
    MONARCH_CUDA_TRY(launch_chained(plane_transpose_kernel<TO_PLANES>, (unsigned)grid, kTrThreads, kTrSmem, s, in.map ? *in.map : out, out, p));
    note_launch();
    return MONARCH_OK;
}

size_t planes_bytes(int64_t tokens) { return (size_t)((tokens + 127) / 128) * 128 * kB * kB * 2; }

}  // namespace
}  // namespace tc

void debug_skip_next_plane_load(long long item) { tc::g_skip_load.store(item); }

// Forward workspace: [status][tile counters 64 KB][u' planes][w' planes]; the backward call reads u' from it.
constexpr size_t kChainCounterBytes = 65536;
size_t chain_fwd_m128_workspace_bytes(int64_t tokens)
{
    return MONARCH_STATUS_BYTES + kChainCounterBytes + 2 * tc::planes_bytes(tokens);
}
namespace tc {
namespace {
// true when chain_fwd_m128 runs as one persistent launch for this many tokens (every CTA resident, counters fit)
bool fwd_runs_fused(int64_t tokens)
{
    int sms = 0;
    if (device_sms(&sms) != MONARCH_OK) return false;
    return chain_fused_enabled() && sms >= kB && (tokens + 127) / 128 <= (int64_t)kFusedCounters;
}
}  // namespace
}  // namespace tc

// u' as either form of the forward pass leaves it: planes [tile][j][k][t]
const void *chain_fwd_m128_saved_u(const void *fwd_ws, int64_t tokens)
{
    (void)tokens;
    return (const char *)fwd_ws + MONARCH_STATUS_BYTES + kChainCounterBytes;
}
// Backward workspace: [status][tile counters 64 KB][dw' planes][du' planes][u' planes (when the forward call's are not passed)]
size_t chain_bwd_m128_workspace_bytes(int64_t tokens)
{
    return MONARCH_STATUS_BYTES + kChainCounterBytes + 3 * tc::planes_bytes(tokens);
}

// y = P L P^T R x (Def. 3.1; Section 3.3 steps 1-3): one persistent launch, or three launches.
int chain_fwd_m128(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws, cudaStream_t s)
{
    using namespace tc;
    if (tokens == 0) return MONARCH_OK;
    if (tokens > (int64_t)1 << 30) return MONARCH_ERR_UNSUPPORTED;
    const int ntiles = (int)((tokens + 127) / 128);
    unsigned *status = (unsigned *)ws;
    char *up = (char *)ws + MONARCH_STATUS_BYTES + kChainCounterBytes, *wp = up + planes_bytes(tokens);
    CUtensorMap mx, my, mR, mL, mu_st, mw_st;
    MONARCH_TRY(map_tokens(&mx, x, tokens));
    MONARCH_TRY(map_weights(&mR, R));
    MONARCH_TRY(map_weights(&mL, L));
    if (fwd_runs_fused(tokens) && g_skip_load.load(std::memory_order_relaxed) < 0) {
        // one persistent launch; every CTA must be resident at once (one per SM)
        MONARCH_CUDA_TRY(cudaFuncSetAttribute(chain_fused_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem));
        FusedParams fp;
        fp.status = status;
        fp.cnt1 = (unsigned *)((char *)ws + MONARCH_STATUS_BYTES);
        fp.cnt2 = fp.cnt1 + kFusedCounters;
        fp.ntiles = ntiles;
        fp.u = up;
        fp.w = wp;
        fp.y = (char *)y;
        fp.x = (const char *)x;
        fp.tokens = tokens;
        fp.trace = nullptr;
#ifdef MONARCH_TRACE
        if (const char *e = getenv("MONARCH_TRACE_PTR")) fp.trace = (long long *)strtoull(e, nullptr, 0);
#endif
        MONARCH_CUDA_TRY(launch_chained(chain_fused_fwd_kernel, kB, kFusedThreads, kFusedSmem, s, mx, mR, mL, fp));
        note_launch();
        return MONARCH_OK;
    }
    MONARCH_TRY(map_tokens(&my, y, tokens));
    MONARCH_TRY(map_pieces(&mu_st, up, ntiles));
    MONARCH_TRY(map_pieces(&mw_st, wp, ntiles));
    // step 1 + inner permutation: D_k[j][t] = sum_i R[k][j][i] x[t][k*128+i]  ->  pieces of u' (row j to consumer j)
    MONARCH_TRY((launch_gemm<kLdX, true, false, false, kStP, false, kLdX, false, true>({&mx, nullptr}, {nullptr, nullptr}, mR, mu_st, nullptr,
                                                                                          ntiles, status, s)));
    // step 2: D_j[l][t] = sum_k L[j][l][k] u'_j[k][t]  ->  pieces of w' (row l to consumer l)
    MONARCH_TRY((launch_gemm<kLdC, true, false, true, kStP, false, kLdX, false, true>({nullptr, up}, {nullptr, nullptr}, mL, mw_st, nullptr,
                                                                                         ntiles, status, s, 0, 1)));
    // step 3 (outer permutation): y[t][l*128+j] = w'_l[j][t]
    return launch_transpose<false>({nullptr, wp}, my, ntiles, status, s);
}

// dx = M^T dy, dL, dR (the adjoints of steps 1-3); saved_up = u' of the forward call or null (recomputed).
// accumulate = 0: dL and dR are overwritten (every block of them has one writing CTA), 1: added to.
int chain_bwd_m128(const void *x, const void *dy, const void *L, const void *R, const void *saved_up, void *dx, float *dL,
                   float *dR, int accumulate, int want_dx, int want_dw, int64_t tokens, void *ws, cudaStream_t s)
{
    using namespace tc;
    if (tokens == 0) return MONARCH_OK;
    if (tokens > (int64_t)1 << 30) return MONARCH_ERR_UNSUPPORTED;
    const int ntiles = (int)((tokens + 127) / 128);
    unsigned *status = (unsigned *)ws;
    char *dwp = (char *)ws + MONARCH_STATUS_BYTES + kChainCounterBytes, *dup = dwp + planes_bytes(tokens),
         *up_own = dup + planes_bytes(tokens);
    CUtensorMap mx, mdy, mdx, mR, mL, mdw_st, mdu_st, mu_st;
    MONARCH_TRY(map_tokens(&mdy, dy, tokens));
    MONARCH_TRY(map_weights(&mR, R));
    MONARCH_TRY(map_weights(&mL, L));
    MONARCH_TRY(map_pieces(&mdw_st, dwp, ntiles));
    MONARCH_TRY(map_pieces(&mdu_st, dup, ntiles));
    if (want_dx) MONARCH_TRY(map_tokens(&mdx, dx, tokens));
    else mdx = mdy;
    const char *up = (const char *)saved_up;
    if (want_dw) {
        MONARCH_TRY(map_tokens(&mx, x, tokens));
        if (up == nullptr) {
            MONARCH_TRY(map_pieces(&mu_st, up_own, ntiles));
            MONARCH_TRY((launch_gemm<kLdX, true, false, false, kStP, false, kLdX, false, true>({&mx, nullptr}, {nullptr, nullptr}, mR, mu_st,
                                                                                                  nullptr, ntiles, status, s)));
            up = up_own;
        }
    }
    // Tile order: a launch walks the tiles in the opposite direction of the one before it, so that it starts with what
    // is still in L2 (an intermediate is 134 MB at 4096 tokens, L2 holds 126).
    // dw' (consumer j, producer l): row j of the transposed tile dy[t][l*128 + j]
    MONARCH_TRY(launch_transpose<true>({&mdy, nullptr}, mdw_st, ntiles, status, s));
    // du'_k[j][t] = sum_l L[j][l][k] dw'_j[l][t] -> pieces of du' (row k to consumer k)   (+ dL[j][l][k] += sum_t dw'_j[l][t] u'_j[k][t])
    if (want_dw)
        MONARCH_TRY((launch_gemm<kLdC, true, true, true, kStP, true, kLdC, false, true>({nullptr, dwp}, {nullptr, up}, mL, mdu_st, dL, ntiles,
                                                                                          status, s, !accumulate, 1, 1)));
    else
        MONARCH_TRY((launch_gemm<kLdC, true, true, true, kStP, false, kLdC, false, true>({nullptr, dwp}, {nullptr, nullptr}, mL, mdu_st, nullptr,
                                                                                           ntiles, status, s, 0, 1, 1)));
    // dx[t][k*128+i] = sum_j du'_k[j][t] R[k][j][i]        (+ dR[k][j][i] += sum_t du'_k[j][t] x[t][k*128+i])
    if (want_dw && want_dx)
        return launch_gemm<kLdC, false, true, true, kStX, true, kLdX, true, true>({nullptr, dup}, {&mx, nullptr}, mR, mdx, dR, ntiles, status, s,
                                                                                  !accumulate, 0, 1);
    if (want_dw)
        return launch_gemm<kLdC, false, true, true, kStX, true, kLdX, true, false>({nullptr, dup}, {&mx, nullptr}, mR, mdx, dR, ntiles, status, s,
                                                                                   !accumulate, 0, 1);
    return launch_gemm<kLdC, false, true, true, kStX, false, kLdX, true, true>({nullptr, dup}, {nullptr, nullptr}, mR, mdx, nullptr, ntiles, status, s,
                                                                               0, 0, 1);
}

}  // namespace monarch
