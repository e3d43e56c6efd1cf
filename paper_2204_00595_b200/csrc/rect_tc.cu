// Stage 1 of the general (rectangular) Monarch multiply on the tensor cores, bf16:
//   u[t][k*b + j] = sum_i R[k][j][i] x[t][k*b1 + i]      (appendix: R = diag(R_0 .. R_{q-1}), R_k of size b x b1)
// i.e. q independent GEMMs  U_k [T x b] = X_k [T x b1] R_k^T  whose operands are both K-major as stored.  With few,
// large blocks (q = 4 blocks of 1024 x 1024 for n = 4096) this stage holds nearly all the FLOPs of the multiply
// and is bound by the tensor pipe, not by HBM.
//
// Persistent kernel, one CTA per SM, 128-token x NT-column output tiles (NT = 256, 128 or 64, the widest that
// divides b: a 128 x 256 x 16 MMA keeps the tensor pipe busy for longer than it takes one thread to issue it):
//   warp 4 lane 0   TMA loads of the x tile (128 x 64) and the R_k tile (NT x 64), 128-byte swizzle, ring of kStages
//   warp 5 lane 0   tcgen05.mma M = 128, N = NT, K = 16, four per 64-wide K chunk, accumulators in TMEM,
//                   two accumulator buffers so that the epilogue of one tile overlaps the MMAs of the next
//   warps 0-3       epilogue: TMEM -> registers -> bf16 -> swizzled staging tile (two, alternating) -> one TMA
//                   store per 64 columns
// Rows past the last token are zero-filled on load and clipped on store by the tensor maps.
// The same kernel with BT = true computes the adjoint  dx[t][k*b1 + i] = sum_j R[k][j][i] du[t][k*b + j]:  the
// contraction then runs over the rows of R_k, so the B operand is MN-major (64 x 64 boxes of R_k, 128-byte swizzle,
// atoms 8 KB apart along N, 16 rows of K = 2 KB).
#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

constexpr int kTokTile = 128, kKChunk = 64;
constexpr int kThreads = 6 * 32;

struct RectParams {
    unsigned *status;
    int q, kdim, ndim;                // blocks, contraction length and outputs per block
    int mtiles, ntiles_per_block;     // output tiles: mtiles x (q * ntiles_per_block)
};

constexpr int kMaxStages = 5;
template <int NT> struct RectSmem {
    static constexpr int kStages = NT == 256 ? 4 : kMaxStages;
    static constexpr int kABytes = kTokTile * kKChunk * 2, kBBytes = NT * kKChunk * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kStagingBytes = kTokTile * 128;                       // 64 columns of bf16
    static constexpr int kBytes = kStages * kStageBytes + 2 * kStagingBytes + 1024;
};

struct RectBars {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t acc_full[2], acc_empty[2];
};

template <int NT, bool BT>
__global__ void __launch_bounds__(kThreads, 1)
rect_stage1_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_R,
                   const __grid_constant__ CUtensorMap tm_u, const RectParams p)
{
    using S = RectSmem<NT>;
    constexpr int kStages = S::kStages;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) RectBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead_s;

    const uint32_t ring0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging0 = ring0 + kStages * S::kStageBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *dead = &dead_s;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&bars.acc_full[a]), 1);
            mbar_init(smem_u32(&bars.acc_empty[a]), 4);
        }
        fence_mbar_init();
        dead_s = 0;
        tma_prefetch_desc(&tm_x); tma_prefetch_desc(&tm_R); tma_prefetch_desc(&tm_u);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 2 * NT);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    const int ntiles = p.q * p.ntiles_per_block;
    const long long total = (long long)p.mtiles * ntiles;
    const int kchunks = p.kdim / kKChunk;
    const uint32_t full0 = smem_u32(bars.full), empty0 = smem_u32(bars.empty);
    const uint32_t accf0 = smem_u32(bars.acc_full), acce0 = smem_u32(bars.acc_empty);

    if (warp == 4) {
        // ------------------------------------------------------------ loader
        if (lane == 0) {
            uint32_t n = 0;                                   // chunks loaded so far
            bool ok = true;
            for (long long tile = blockIdx.x; ok && tile < total; tile += gridDim.x) {
                const int mt = (int)(tile / ntiles), nt = (int)(tile % ntiles);
                const int k = nt / p.ntiles_per_block, n0 = (nt % p.ntiles_per_block) * NT;
                for (int c = 0; c < kchunks; ++c, ++n) {
                    const uint32_t s = n % kStages;
                    if (!mbar_wait(empty0 + s * 8, ((n / kStages) & 1) ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
                    mbar_expect_tx(full0 + s * 8, S::kStageBytes);
                    tma_load_2d(ring0 + s * S::kStageBytes, &tm_x, k * p.kdim + c * kKChunk, mt * kTokTile, full0 + s * 8);
                    if constexpr (!BT) {
                        tma_load_2d(ring0 + s * S::kStageBytes + S::kABytes, &tm_R, c * kKChunk, k * p.ndim + n0, full0 + s * 8);
                    } else {
#pragma unroll
                        for (int a = 0; a < NT / 64; ++a)      // 64 (K rows) x 64 (N columns) boxes of R_k
                            tma_load_2d(ring0 + s * S::kStageBytes + S::kABytes + a * 8192, &tm_R, n0 + a * 64,
                                        k * p.kdim + c * kKChunk, full0 + s * 8);
                    }
                }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(kTokTile, NT, 0, BT ? 1 : 0);
            uint32_t n = 0, it = 0;
            bool ok = true;
            for (long long tile = blockIdx.x; ok && tile < total; tile += gridDim.x, ++it) {
                const uint32_t buf = it & 1;
                if (!mbar_wait(acce0 + buf * 8, ((it >> 1) & 1) ^ 1, p.status, dead, kErrTmemWait)) break;
                tc_fence_after();
                const uint32_t d = tmem_base + buf * NT;
                for (int c = 0; c < kchunks; ++c, ++n) {
                    const uint32_t s = n % kStages;
                    if (!mbar_wait(full0 + s * 8, (n / kStages) & 1, p.status, dead, kErrTmaWait)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = ring0 + s * S::kStageBytes;
                    const uint64_t ad = make_smem_desc(a_addr, 16, 1024, kSwizzle128);
                    const uint64_t bd = BT ? make_smem_desc(a_addr + S::kABytes, 8192, 1024, kSwizzle128)
                                           : make_smem_desc(a_addr + S::kABytes, 16, 1024, kSwizzle128);
                    constexpr uint32_t bstep = BT ? 128 : 2;          // 16 of K: 2 KB of rows, or 32 bytes along a row
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_f16_ss(d, ad + 2 * kk, bd + bstep * kk, idesc, (c | kk) != 0);
                    mma_commit(empty0 + s * 8);
                }
                if (!ok) break;
                mma_commit(accf0 + buf * 8);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 0-3 = TMEM lanes 32w..32w+31)
        const int row = warp * 32 + lane;
        uint32_t it = 0, nchunk = 0;                                   // 64-column chunks stored so far
        for (long long tile = blockIdx.x; tile < total; tile += gridDim.x, ++it) {
            const int mt = (int)(tile / ntiles), nt = (int)(tile % ntiles);
            const int k = nt / p.ntiles_per_block, n0 = (nt % p.ntiles_per_block) * NT;
            const uint32_t buf = it & 1;
            if (!mbar_wait(accf0 + buf * 8, (it >> 1) & 1, p.status, dead, kErrMmaWait)) break;
            tc_fence_after();
#pragma unroll 1
            for (int h = 0; h < NT / 64; ++h, ++nchunk) {
                const uint32_t stg = staging0 + (nchunk & 1) * S::kStagingBytes;
                // this staging tile is free once the store issued two chunks ago has read it
                if (threadIdx.x == 0) tma_store_wait_read<1>();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + buf * NT + h * 64;
                uint32_t v[4][16];
#pragma unroll
                for (int i = 0; i < 4; ++i) tmem_ld16(taddr + i * 16, v[i]);
                tmem_ld_wait();
                if (h == NT / 64 - 1) {
                    // accumulator buffer drained: hand it back to the MMA warp
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
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + ((c ^ (row & 7)) << 4)),
                                 "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                }
                fence_proxy_async_smem();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (threadIdx.x == 0) {
                    tma_store_2d(&tm_u, stg, k * p.ndim + n0 + h * 64, mt * kTokTile);
                    tma_store_commit();
                }
            }
        }
        if (threadIdx.x == 0) tma_store_wait_all<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 2 * NT);
}

// ---------------------------------------------------------------------------------------------------------
// The same stage on CTA pairs (clusters of two, tcgen05 cta_group::2): one MMA instruction of 256 x 256 x 16 runs on
// both SMs.  Each CTA loads the x rows of its own 128 tokens and HALF of the 256 weight rows of the tile (its
// N/2 rows of the B operand), so the weight traffic from L2 to shared memory halves and the ring gets deeper; each
// CTA ends up with the 128 x 256 accumulator of its own tokens in its own TMEM, laid out as for a single CTA, and
// the epilogue is unchanged.  The even CTA's MMA thread issues for both; both CTAs' TMA loads count their bytes on
// the even CTA's "stage full" barrier (a software relay of "my half has landed" through a release-arrive on the
// peer's barrier cost about a microsecond per stage and made the kernel 2.5x slower).  Freed ring slots and finished
// accumulators are announced to both CTAs by a multicast commit; drained accumulators are reported back to the
// even CTA.
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = 2 * kTokTile * kKChunk * 2;                // A 16 KB + this CTA's half of B 16 KB
constexpr int kPairSmem = kPairStages * kPairStageBytes + 2 * (kTokTile * 128) + 1024;

struct PairBars {
    uint64_t full[kPairStages], empty[kPairStages];                     // full: used in the even CTA only
    uint64_t acc_full[2], acc_empty[2];
};

template <bool BT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
rect_stage1_pair_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_R,
                        const __grid_constant__ CUtensorMap tm_u, const RectParams p)
{
    constexpr int NT = 256;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) PairBars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead_s;

    const uint32_t ring0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging0 = ring0 + kPairStages * kPairStageBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    volatile int *dead = &dead_s;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);                        // the even CTA's expect_tx arrival
            mbar_init(smem_u32(&bars.empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&bars.acc_full[a]), 1);
            mbar_init(smem_u32(&bars.acc_empty[a]), 8);                   // four epilogue warps of each CTA
        }
        fence_mbar_init();
        dead_s = 0;
        tma_prefetch_desc(&tm_x); tma_prefetch_desc(&tm_R); tma_prefetch_desc(&tm_u);
    }
    if (warp == 0) {
        tmem_alloc_pair(smem_u32(&tmem_base_s), 2 * NT);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_arrive_release();                                             // both CTAs' barriers exist before any remote arrive
    cluster_wait_acquire();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    const int ntiles = p.q * p.ntiles_per_block;
    const int mpairs = (p.mtiles + 1) / 2;                                // token tiles come in pairs, one per CTA
    const long long total = (long long)mpairs * ntiles;
    const int kchunks = p.kdim / kKChunk;
    const uint32_t full0 = smem_u32(bars.full), empty0 = smem_u32(bars.empty);
    const uint32_t accf0 = smem_u32(bars.acc_full), acce0 = smem_u32(bars.acc_empty);

    if (warp == 4) {
        // ------------------------------------------------------------ loader (both CTAs)
        if (lane == 0) {
            uint32_t n = 0;
            bool ok = true;
            for (long long tile = pair; ok && tile < total; tile += npairs) {
                const int mt = (int)(tile / ntiles) * 2 + (int)rank, nt = (int)(tile % ntiles);
                const int k = nt / p.ntiles_per_block, n0 = (nt % p.ntiles_per_block) * NT;
                for (int c = 0; c < kchunks; ++c, ++n) {
                    const uint32_t s = n % kPairStages;
                    if (!mbar_wait(empty0 + s * 8, ((n / kPairStages) & 1) ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
                    // the even CTA announces the bytes of both halves; either CTA's may land first
                    if (rank == 0) mbar_expect_tx(full0 + s * 8, 2 * kPairStageBytes);
                    tma_load_2d_pair(ring0 + s * kPairStageBytes, &tm_x, k * p.kdim + c * kKChunk, mt * kTokTile, full0 + s * 8);
                    if constexpr (!BT) {
                        tma_load_2d_pair(ring0 + s * kPairStageBytes + kPairStageBytes / 2, &tm_R, c * kKChunk,
                                         k * p.ndim + n0 + (int)rank * (NT / 2), full0 + s * 8);
                    } else {
#pragma unroll
                        for (int a = 0; a < 2; ++a)          // this CTA's 128 columns of R_k: two 64 x 64 boxes
                            tma_load_2d_pair(ring0 + s * kPairStageBytes + kPairStageBytes / 2 + a * 8192, &tm_R,
                                             n0 + (int)rank * (NT / 2) + a * 64, k * p.kdim + c * kKChunk, full0 + s * 8);
                    }
                }
            }
        }
    } else if (warp == 5) {
        if (lane == 0 && rank == 0) {
            // ------------------------------------------------------------ even CTA: MMA issuer for the pair
            constexpr uint32_t idesc = make_idesc_bf16(2 * kTokTile, NT, 0, BT ? 1 : 0);
            constexpr uint32_t bstep = BT ? 128 : 2;
            uint32_t n = 0, it = 0;
            bool ok = true;
            for (long long tile = pair; ok && tile < total; tile += npairs, ++it) {
                const uint32_t buf = it & 1;
                if (!mbar_wait<true>(acce0 + buf * 8, ((it >> 1) & 1) ^ 1, p.status, dead, kErrTmemWait)) break;
                tc_fence_after();
                const uint32_t d = tmem_base + buf * NT;
                for (int c = 0; c < kchunks; ++c, ++n) {
                    const uint32_t s = n % kPairStages;
                    if (!mbar_wait<true>(full0 + s * 8, (n / kPairStages) & 1, p.status, dead, kErrTmaWait)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = ring0 + s * kPairStageBytes;
                    const uint64_t ad = make_smem_desc(a_addr, 16, 1024, kSwizzle128);
                    const uint64_t bd = BT ? make_smem_desc(a_addr + kPairStageBytes / 2, 8192, 1024, kSwizzle128)
                                           : make_smem_desc(a_addr + kPairStageBytes / 2, 16, 1024, kSwizzle128);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_f16_ss_pair(d, ad + 2 * kk, bd + bstep * kk, idesc, (c | kk) != 0);
                    mma_commit_pair(empty0 + s * 8, 3);
                }
                if (!ok) break;
                mma_commit_pair(accf0 + buf * 8, 3);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (both CTAs; own 128 tokens)
        const int row = warp * 32 + lane;
        const uint32_t acce_leader = map_to_cta(acce0, 0);
        uint32_t it = 0, nchunk = 0;
        for (long long tile = pair; tile < total; tile += npairs, ++it) {
            const int mt = (int)(tile / ntiles) * 2 + (int)rank, nt = (int)(tile % ntiles);
            const int k = nt / p.ntiles_per_block, n0 = (nt % p.ntiles_per_block) * NT;
            const uint32_t buf = it & 1;
            if (!mbar_wait(accf0 + buf * 8, (it >> 1) & 1, p.status, dead, kErrMmaWait)) break;
            tc_fence_after();
#pragma unroll 1
            for (int h = 0; h < NT / 64; ++h, ++nchunk) {
                const uint32_t stg = staging0 + (nchunk & 1) * (kTokTile * 128);
                if (threadIdx.x == 0) tma_store_wait_read<1>();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + buf * NT + h * 64;
                uint32_t v[4][16];
#pragma unroll
                for (int i = 0; i < 4; ++i) tmem_ld16(taddr + i * 16, v[i]);
                tmem_ld_wait();
                if (h == NT / 64 - 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_remote(acce_leader + buf * 8);
                }
                const uint32_t dst = stg + row * 128;
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
                fence_proxy_async_smem();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (threadIdx.x == 0) {
                    tma_store_2d(&tm_u, stg, k * p.ndim + n0 + h * 64, mt * kTokTile);
                    tma_store_commit();
                }
            }
        }
        if (threadIdx.x == 0) tma_store_wait_all<0>();
    }

    // the even CTA's barriers receive arrivals from the odd CTA until it is done: leave together
    tc_fence_before();
    __syncthreads();
    cluster_arrive_release();
    cluster_wait_acquire();
    if (warp == 0) tmem_dealloc_pair(tmem_base, 2 * NT);
}

template <bool BT>
int launch_pair(const void *in, const void *W, void *out, int64_t tokens, int q, int kdim, int ndim, unsigned *status,
                cudaStream_t s, bool *used)
{
    *used = false;
    CUtensorMap tm_x, tm_R, tm_u;
    MONARCH_TRY(encode_tmap_2d(&tm_x, in, (uint64_t)tokens, (uint64_t)q * kdim, (uint64_t)q * kdim * 2, kTokTile, kKChunk, 128));
    if (BT)
        MONARCH_TRY(encode_tmap_2d(&tm_R, W, (uint64_t)q * kdim, (uint64_t)ndim, (uint64_t)ndim * 2, 64, 64, 128));
    else
        MONARCH_TRY(encode_tmap_2d(&tm_R, W, (uint64_t)q * ndim, (uint64_t)kdim, (uint64_t)kdim * 2, 128, kKChunk, 128));
    MONARCH_TRY(encode_tmap_2d(&tm_u, out, (uint64_t)tokens, (uint64_t)q * ndim, (uint64_t)q * ndim * 2, kTokTile, 64, 128));
    static PerDeviceCache max_pairs_cache;
    int max_pairs = max_pairs_cache.get();
    if (max_pairs < 0) {
        MONARCH_CUDA_TRY(cudaFuncSetAttribute(rect_stage1_pair_kernel<BT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmem));
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2, 1, 1);
        cfg.blockDim = dim3(kThreads, 1, 1);
        cfg.dynamicSmemBytes = kPairSmem;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, rect_stage1_pair_kernel<BT>, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
        max_pairs = n;
        max_pairs_cache.set(n);
    }
    if (max_pairs < 1) return MONARCH_OK;                                 // the caller falls back to single CTAs
    RectParams p;
    p.status = status;
    p.q = q; p.kdim = kdim; p.ndim = ndim;
    p.mtiles = (int)((tokens + kTokTile - 1) / kTokTile);
    p.ntiles_per_block = ndim / 256;
    const long long total = (long long)((p.mtiles + 1) / 2) * q * p.ntiles_per_block;
    const int pairs = (int)(total < max_pairs ? total : max_pairs);
    rect_stage1_pair_kernel<BT><<<2 * pairs, kThreads, kPairSmem, s>>>(tm_x, tm_R, tm_u, p);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    *used = true;
    return MONARCH_OK;
}

// in: [tokens][q * kdim], W: [q][b][b1] (kdim = b1, ndim = b) or, with BT, contracted over its rows (kdim = b, ndim = b1)
template <int NT, bool BT>
int launch(const void *in, const void *W, void *out, int64_t tokens, int q, int kdim, int ndim, unsigned *status,
           cudaStream_t s)
{
    using S = RectSmem<NT>;
    CUtensorMap tm_x, tm_R, tm_u;
    MONARCH_TRY(encode_tmap_2d(&tm_x, in, (uint64_t)tokens, (uint64_t)q * kdim, (uint64_t)q * kdim * 2, kTokTile, kKChunk, 128));
    if (BT)
        MONARCH_TRY(encode_tmap_2d(&tm_R, W, (uint64_t)q * kdim, (uint64_t)ndim, (uint64_t)ndim * 2, 64, 64, 128));
    else
        MONARCH_TRY(encode_tmap_2d(&tm_R, W, (uint64_t)q * ndim, (uint64_t)kdim, (uint64_t)kdim * 2, NT, kKChunk, 128));
    MONARCH_TRY(encode_tmap_2d(&tm_u, out, (uint64_t)tokens, (uint64_t)q * ndim, (uint64_t)q * ndim * 2, kTokTile, 64, 128));
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    static bool attr = false;
    if (!attr) {
        MONARCH_CUDA_TRY(cudaFuncSetAttribute(rect_stage1_kernel<NT, BT>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kBytes));
        attr = true;
    }
    RectParams p;
    p.status = status;
    p.q = q; p.kdim = kdim; p.ndim = ndim;
    p.mtiles = (int)((tokens + kTokTile - 1) / kTokTile);
    p.ntiles_per_block = ndim / NT;
    const long long total = (long long)p.mtiles * q * p.ntiles_per_block;
    const int grid = (int)(total < sms ? total : sms);
    rect_stage1_kernel<NT, BT><<<grid, kThreads, S::kBytes, s>>>(tm_x, tm_R, tm_u, p);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

// ---------------------------------------------------------------------------------------------------------
// Stage 2 when L's blocks are at most 4 x 4:  y[t][l*b + j] = sum_k Lp[j][l][k] u[t][k*b + j]  as a streaming pass.
// A CTA owns 256 columns j and a slab of tokens; TMA brings 16-token tiles of the q slices u[t][k*b + j0 ..] into a
// three-stage ring (no thread holds a load in flight, so the pass is not limited by registers x occupancy), the
// blocks sit in shared memory as fp32, and each thread turns 8 columns of two tokens into r x 8 outputs per step,
// written back with 16-byte stores (a warp writes 512 contiguous bytes of a slice y[t][l*b + .]).
constexpr int kS2Cols = 256, kS2Tok = 16, kS2Stages = 3, kS2Threads = 256;
constexpr int kS2SliceBytes = kS2Tok * kS2Cols * 2;                 // one k slice of a tile
constexpr int kS2SmemBytes = kS2Stages * 4 * kS2SliceBytes + 128;     // two CTAs per SM with the 16 KB of blocks

__device__ __forceinline__ float4 lds128f(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds128u(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ float bf_elem(const uint4 &v, int e)
{
    const uint32_t w = e < 2 ? v.x : e < 4 ? v.y : e < 6 ? v.z : v.w;
    return (e & 1) ? __uint_as_float(w & 0xFFFF0000u) : __uint_as_float(w << 16);
}

__global__ void __launch_bounds__(kS2Threads, 2)
rect_stage2_stream_kernel(const __grid_constant__ CUtensorMap tm_u, const __nv_bfloat16 *__restrict__ Lp,
                          __nv_bfloat16 *__restrict__ y, unsigned *status, long long tokens, int q, int b, int r,
                          int tokens_per_slab, int wt)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ float4 ws[4][4][2][32];            // [l][k][half][lane]: columns 8 lane + 4 half + (0..3)
    __shared__ __align__(8) uint64_t full[kS2Stages];
    __shared__ int dead_s;
    const uint32_t ring0 = (smem_u32(smem_raw) + 127u) & ~127u;
    const int j0 = blockIdx.x * kS2Cols;
    volatile int *dead = &dead_s;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kS2Stages; ++s) mbar_init(smem_u32(&full[s]), 1);
        fence_mbar_init();
        dead_s = 0;
        tma_prefetch_desc(&tm_u);
    }
    for (int i = threadIdx.x; i < 16 * kS2Cols; i += kS2Threads) {
        const int jl = i >> 4, l = (i >> 2) & 3, k = i & 3;
        float v = 0.0f;
        // wt: the blocks are stored [j][k][l] (the adjoint pass reads L's blocks transposed)
        if (j0 + jl < b && l < r && k < q) v = __bfloat162float(Lp[(size_t)(j0 + jl) * r * q + (wt ? k * r + l : l * q + k)]);
        reinterpret_cast<float *>(&ws[l][k][(jl >> 2) & 1][jl >> 3])[jl & 3] = v;
    }
    __syncthreads();

    const long long t0 = (long long)blockIdx.y * tokens_per_slab;
    const long long t1 = t0 + tokens_per_slab < tokens ? t0 + tokens_per_slab : tokens;
    const int ntiles = t1 > t0 ? (int)((t1 - t0 + kS2Tok - 1) / kS2Tok) : 0;
    const uint32_t full0 = smem_u32(full);
    const uint32_t stage_bytes = (uint32_t)q * kS2SliceBytes;

    auto issue = [&](int tile) {
        const uint32_t s = tile % kS2Stages;
        mbar_expect_tx(full0 + s * 8, stage_bytes);
        for (int k = 0; k < q; ++k)
            tma_load_2d(ring0 + s * 4 * kS2SliceBytes + k * kS2SliceBytes, &tm_u, k * b + j0,
                        (int)(t0 + (long long)tile * kS2Tok), full0 + s * 8);
    };
    if (threadIdx.x == 0)
        for (int tile = 0; tile < kS2Stages - 1 && tile < ntiles; ++tile) issue(tile);

    const int lane = threadIdx.x & 31, tr = threadIdx.x >> 5;             // 32 threads per token row, rows tr, tr + 8
    const bool active = j0 + lane * 8 < b;
    const uint32_t ws0 = smem_u32(ws);
    for (int tile = 0; tile < ntiles; ++tile) {
        // the stage this load goes to was read in the previous step, which ended with a CTA barrier
        if (threadIdx.x == 0 && tile + kS2Stages - 1 < ntiles) issue(tile + kS2Stages - 1);
        const uint32_t s = tile % kS2Stages;
        if (!mbar_wait(full0 + s * 8, (tile / kS2Stages) & 1, status, dead, kErrTmaWait)) break;
        const long long ta = t0 + (long long)tile * kS2Tok + tr, tb = ta + 8;
        if (active && ta < t1) {
            const bool two = tb < t1;
            const uint32_t src = ring0 + s * 4 * kS2SliceBytes + lane * 16;
            uint4 v[2][4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                v[0][k] = k < q ? lds128u(src + k * kS2SliceBytes + tr * (kS2Cols * 2)) : make_uint4(0u, 0u, 0u, 0u);
                v[1][k] = k < q ? lds128u(src + k * kS2SliceBytes + (tr + 8) * (kS2Cols * 2)) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll 1
            for (int l = 0; l < r; ++l) {
                float acc[2][8];
#pragma unroll
                for (int tt = 0; tt < 2; ++tt)
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[tt][e] = 0.0f;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float4 wa = lds128f(ws0 + ((l * 4 + k) * 2 + 0) * 512 + lane * 16);
                    const float4 wb = lds128f(ws0 + ((l * 4 + k) * 2 + 1) * 512 + lane * 16);
                    const float wv[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
                    for (int tt = 0; tt < 2; ++tt)
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[tt][e] = fmaf(wv[e], bf_elem(v[tt][k], e), acc[tt][e]);
                }
#pragma unroll
                for (int tt = 0; tt < 2; ++tt) {
                    if (tt == 1 && !two) break;
                    const uint4 o = make_uint4(pack_bf16(acc[tt][0], acc[tt][1]), pack_bf16(acc[tt][2], acc[tt][3]),
                                               pack_bf16(acc[tt][4], acc[tt][5]), pack_bf16(acc[tt][6], acc[tt][7]));
                    *reinterpret_cast<uint4 *>(y + (size_t)(tt ? tb : ta) * r * b + (size_t)l * b + j0 + lane * 8) = o;
                }
            }
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------------------
// dL[j][l][k] += sum_t dy[t][l*b + j] u[t][k*b + j] for blocks of at most 4 x 4, as a streaming pass like the one
// above: TMA brings 16-token tiles of the r slices of dy and the q slices of u into a three-stage ring; a thread owns
// 8 columns and keeps their r x q x 8 partial sums in registers (one CTA per SM), adding them to dL at the end.
__global__ void __launch_bounds__(kS2Threads, 1)
rect_dl_stream_kernel(const __grid_constant__ CUtensorMap tm_dy, const __grid_constant__ CUtensorMap tm_u,
                      float *__restrict__ dL, unsigned *status, long long tokens, int q, int b, int r, int tokens_per_slab)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full[kS2Stages];
    __shared__ int dead_s;
    const uint32_t ring0 = (smem_u32(smem_raw) + 127u) & ~127u;
    const int j0 = blockIdx.x * kS2Cols;
    volatile int *dead = &dead_s;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kS2Stages; ++s) mbar_init(smem_u32(&full[s]), 1);
        fence_mbar_init();
        dead_s = 0;
        tma_prefetch_desc(&tm_dy);
        tma_prefetch_desc(&tm_u);
    }
    __syncthreads();
    const long long t0 = (long long)blockIdx.y * tokens_per_slab;
    const long long t1 = t0 + tokens_per_slab < tokens ? t0 + tokens_per_slab : tokens;
    const int ntiles = t1 > t0 ? (int)((t1 - t0 + kS2Tok - 1) / kS2Tok) : 0;
    const uint32_t full0 = smem_u32(full);
    const uint32_t stage_bytes = (uint32_t)(q + r) * kS2SliceBytes;
    auto issue = [&](int tile) {
        const uint32_t s = tile % kS2Stages;
        const int row = (int)(t0 + (long long)tile * kS2Tok);
        mbar_expect_tx(full0 + s * 8, stage_bytes);
        for (int l = 0; l < r; ++l)
            tma_load_2d(ring0 + (s * 8 + l) * kS2SliceBytes, &tm_dy, l * b + j0, row, full0 + s * 8);
        for (int k = 0; k < q; ++k)
            tma_load_2d(ring0 + (s * 8 + 4 + k) * kS2SliceBytes, &tm_u, k * b + j0, row, full0 + s * 8);
    };
    if (threadIdx.x == 0)
        for (int tile = 0; tile < kS2Stages - 1 && tile < ntiles; ++tile) issue(tile);

    const int lane = threadIdx.x & 31, tr = threadIdx.x >> 5;
    const bool active = j0 + lane * 8 < b;
    float gsum[4][4][8];
#pragma unroll
    for (int l = 0; l < 4; ++l)
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
            for (int e = 0; e < 8; ++e) gsum[l][k][e] = 0.0f;
    for (int tile = 0; tile < ntiles; ++tile) {
        if (threadIdx.x == 0 && tile + kS2Stages - 1 < ntiles) issue(tile + kS2Stages - 1);
        const uint32_t s = tile % kS2Stages;
        if (!mbar_wait(full0 + s * 8, (tile / kS2Stages) & 1, status, dead, kErrTmaWait)) break;
        const long long ta = t0 + (long long)tile * kS2Tok + tr;
        if (active) {
            const uint32_t src = ring0 + s * 8 * kS2SliceBytes + lane * 16;
#pragma unroll
            for (int tt = 0; tt < 2; ++tt) {
                if (ta + 8 * tt >= t1) break;                     // rows of the next slab, or past the last token
                const uint32_t rowoff = (tr + 8 * tt) * (kS2Cols * 2);
                float gf[4][8];
#pragma unroll
                for (int l = 0; l < 4; ++l) {
                    const uint4 g = l < r ? lds128u(src + l * kS2SliceBytes + rowoff) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                    for (int e = 0; e < 8; ++e) gf[l][e] = bf_elem(g, e);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (k >= q) break;
                    const uint4 uv = lds128u(src + (4 + k) * kS2SliceBytes + rowoff);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float uf = bf_elem(uv, e);
#pragma unroll
                        for (int l = 0; l < 4; ++l) gsum[l][k][e] = fmaf(gf[l][e], uf, gsum[l][k][e]);
                    }
                }
            }
        }
        __syncthreads();
    }
    // the eight token rows of a lane hold partial sums of the same entries: add them up through the (now idle) ring
    // before going to memory - one atomic per entry and CTA instead of eight
    float *red = reinterpret_cast<float *>(smem_raw + (ring0 - smem_u32(smem_raw)));     // [tr][128 entries][32 lanes]
#pragma unroll
    for (int l = 0; l < 4; ++l)
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
            for (int e = 0; e < 8; ++e) red[(tr * 128 + (l * 4 + k) * 8 + e) * 32 + lane] = gsum[l][k][e];
    __syncthreads();
    if (ntiles > 0) {
        for (int i = threadIdx.x; i < 128 * 32; i += kS2Threads) {
            const int ent = i >> 5, ln = i & 31;                    // entry (l, k, e) of lane ln's columns
            const int l = ent >> 5, k = (ent >> 3) & 3, e = ent & 7;
            const int j = j0 + ln * 8 + e;
            if (j < b && l < r && k < q) {
                float sum = 0.0f;
#pragma unroll
                for (int w = 0; w < 8; ++w) sum += red[(w * 128 + ent) * 32 + ln];
                atomicAdd(dL + ((size_t)j * r + l) * q + k, sum);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------------------
// dR[k][j][i] += sum_t du[t][k*b + j] x[t][k*b1 + i]: per block a GEMM whose contraction runs over the tokens, so both
// operands are read token-major (MN-major descriptors over 64-token x 64-column boxes, 128-byte swizzle).  A CTA owns
// a 128 (j) x NT (i) tile of one block's gradient and a slice of the token chunks; its fp32 partial sums go to the
// output with vector reductions in L2.
constexpr int kWgStages = 4;
struct WgParams {
    float *out;
    unsigned *status;
    int q, b, b1, chunks, slices;
    int jtiles, itiles;
};

template <int NT>
__global__ void __launch_bounds__(kThreads, 1)
rect_wgrad_kernel(const __grid_constant__ CUtensorMap tm_du, const __grid_constant__ CUtensorMap tm_x, const WgParams p)
{
    constexpr int kABytes = 2 * 8192, kBBytes = (NT / 64) * 8192, kStageBytes = kABytes + kBBytes;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kWgStages], bar_empty[kWgStages], bar_acc;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead_s;
    const uint32_t ring0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *dead = &dead_s;
    int tile = blockIdx.x;
    const int it = tile % p.itiles; tile /= p.itiles;
    const int jt = tile % p.jtiles;
    const int k = tile / p.jtiles;
    const int j0 = jt * 128, i0 = it * NT;
    const int first = blockIdx.y;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kWgStages; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc), 1);
        fence_mbar_init();
        dead_s = 0;
        tma_prefetch_desc(&tm_du);
        tma_prefetch_desc(&tm_x);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), NT);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    const uint32_t full0 = smem_u32(bar_full), empty0 = smem_u32(bar_empty), acc = smem_u32(&bar_acc);

    if (first < p.chunks) {
        if (warp == 4) {
            if (lane == 0) {
                uint32_t n = 0;
                for (int c = first; c < p.chunks; c += p.slices, ++n) {
                    const uint32_t s = n % kWgStages;
                    if (!mbar_wait(empty0 + s * 8, ((n / kWgStages) & 1) ^ 1, p.status, dead, kErrSlotWait)) break;
                    const uint32_t dst = ring0 + s * kStageBytes, full = full0 + s * 8;
                    mbar_expect_tx(full, kStageBytes);
                    tma_load_2d(dst, &tm_du, k * p.b + j0, c * 64, full);
                    tma_load_2d(dst + 8192, &tm_du, k * p.b + j0 + 64, c * 64, full);
#pragma unroll
                    for (int a = 0; a < NT / 64; ++a)
                        tma_load_2d(dst + kABytes + a * 8192, &tm_x, k * p.b1 + i0 + a * 64, c * 64, full);
                }
            }
        } else if (warp == 5) {
            if (lane == 0) {
                constexpr uint32_t idesc = make_idesc_bf16(128, NT, 1, 1);
                // 64-column swizzle atoms 8 KB apart along M (N); 8-token groups 1 KB apart along K
                const uint64_t desc = make_smem_desc(0, 8192, 1024, kSwizzle128);
                uint32_t n = 0;
                bool ok = true;
                for (int c = first; c < p.chunks; c += p.slices, ++n) {
                    const uint32_t s = n % kWgStages;
                    if (!mbar_wait(full0 + s * 8, (n / kWgStages) & 1, p.status, dead, kErrTmaWait)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t ad = desc | (uint64_t)((ring0 + s * kStageBytes) >> 4);
                    const uint64_t bd = ad + (kABytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)                      // 16 tokens = 2 KB further
                        mma_f16_ss(tmem_base, ad + 128 * kk, bd + 128 * kk, idesc, (n | kk) != 0);
                    mma_commit(empty0 + s * 8);
                }
                if (ok) mma_commit(acc);
            }
        } else {
            if (mbar_wait(acc, 0, p.status, dead, kErrMmaWait)) {
                tc_fence_after();
                const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
                float *out = p.out + ((size_t)k * p.b + j0 + warp * 32 + lane) * p.b1 + i0;
#pragma unroll 1
                for (int c = 0; c < NT; c += 16) {
                    uint32_t v[16];
                    tmem_ld16(lane_base + c, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(out + c + e * 4),
                                     "f"(__uint_as_float(v[e * 4])), "f"(__uint_as_float(v[e * 4 + 1])),
                                     "f"(__uint_as_float(v[e * 4 + 2])), "f"(__uint_as_float(v[e * 4 + 3]))
                                     : "memory");
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, NT);
}

template <int NT>
int launch_wgrad(const void *du, const void *x, float *dR, int64_t tokens, int q, int b1, int b, unsigned *status,
                 cudaStream_t s)
{
    constexpr int smem = kWgStages * (2 * 8192 + (NT / 64) * 8192) + 1024;
    CUtensorMap tm_du, tm_x;
    MONARCH_TRY(encode_tmap_2d(&tm_du, du, (uint64_t)tokens, (uint64_t)q * b, (uint64_t)q * b * 2, 64, 64, 128));
    MONARCH_TRY(encode_tmap_2d(&tm_x, x, (uint64_t)tokens, (uint64_t)q * b1, (uint64_t)q * b1 * 2, 64, 64, 128));
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(rect_wgrad_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    WgParams p;
    p.out = dR;
    p.status = status;
    p.q = q; p.b = b; p.b1 = b1;
    p.chunks = (int)((tokens + 63) / 64);
    p.jtiles = b / 128;
    p.itiles = b1 / NT;
    const long long tiles = (long long)q * p.jtiles * p.itiles;
    long long slices = sms / tiles;
    if (slices < 1) slices = 1;
    if (slices > p.chunks) slices = p.chunks;
    if (tiles > 0x7fffffffLL || slices > 65535) return MONARCH_ERR_UNSUPPORTED;
    p.slices = (int)slices;
    rect_wgrad_kernel<NT><<<dim3((unsigned)tiles, (unsigned)slices), kThreads, smem, s>>>(tm_du, tm_x, p);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

}  // namespace
}  // namespace tc

bool rect_stage1_tc_available(int q, int b1, int b, int dtype)
{
    (void)q;
    return dtype == MONARCH_BF16 && b1 % 64 == 0 && b % 64 == 0;
}

bool rect_stage2_stream_available(int q, int b, int r, int dtype)
{
    return dtype == MONARCH_BF16 && q <= 4 && r <= 4 && b % 8 == 0 && b >= 256;     // a 256-column box fits a slice
}

int rect_stage2_stream(const void *u, const void *Lp, void *y, int64_t tokens, int q, int b, int r, int wt,
                       unsigned *status, cudaStream_t s)
{
    using namespace tc;
    if (tokens == 0) return MONARCH_OK;
    CUtensorMap tm_u;
    MONARCH_TRY(encode_tmap_2d(&tm_u, u, (uint64_t)tokens, (uint64_t)q * b, (uint64_t)q * b * 2, kS2Tok, kS2Cols, 0));
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(rect_stage2_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          kS2SmemBytes));
    const int cx = (b + kS2Cols - 1) / kS2Cols;
    long long slabs = (2LL * sms + cx - 1) / cx;                     // two CTAs per SM, one wave
    if (slabs > (tokens + kS2Tok - 1) / kS2Tok) slabs = (tokens + kS2Tok - 1) / kS2Tok;
    long long per = (tokens + slabs - 1) / slabs;
    per = (per + kS2Tok - 1) / kS2Tok * kS2Tok;
    slabs = (tokens + per - 1) / per;
    if (slabs > 65535) return MONARCH_ERR_UNSUPPORTED;
    rect_stage2_stream_kernel<<<dim3((unsigned)cx, (unsigned)slabs), kS2Threads, kS2SmemBytes, s>>>(
        tm_u, (const __nv_bfloat16 *)Lp, (__nv_bfloat16 *)y, status, tokens, q, b, r, (int)per, wt);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

int rect_stage1_tc(const void *x, const void *R, void *u, int64_t tokens, int q, int b1, int b, unsigned *status,
                   cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    if (b % 256 == 0 && tokens > 128) {
        // two or more token tiles: CTA pairs (falls through where no cluster of two can be resident)
        bool used = false;
        MONARCH_TRY(tc::launch_pair<false>(x, R, u, tokens, q, b1, b, status, s, &used));
        if (used) return MONARCH_OK;
    }
    if (b % 256 == 0) return tc::launch<256, false>(x, R, u, tokens, q, b1, b, status, s);
    return b % 128 == 0 ? tc::launch<128, false>(x, R, u, tokens, q, b1, b, status, s)
                        : tc::launch<64, false>(x, R, u, tokens, q, b1, b, status, s);
}

// dL as a TMA-fed streaming pass: same sizes as the streaming stage 2
int rect_dl_stream(const void *dy, const void *u, float *dL, int64_t tokens, int q, int b, int r, unsigned *status,
                   cudaStream_t s)
{
    using namespace tc;
    if (tokens == 0) return MONARCH_OK;
    CUtensorMap tm_dy, tm_u;
    MONARCH_TRY(encode_tmap_2d(&tm_dy, dy, (uint64_t)tokens, (uint64_t)r * b, (uint64_t)r * b * 2, kS2Tok, kS2Cols, 0));
    MONARCH_TRY(encode_tmap_2d(&tm_u, u, (uint64_t)tokens, (uint64_t)q * b, (uint64_t)q * b * 2, kS2Tok, kS2Cols, 0));
    constexpr int smem = kS2Stages * 8 * kS2SliceBytes + 128;
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(rect_dl_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    const int cx = (b + kS2Cols - 1) / kS2Cols;
    long long slabs = (sms + cx - 1) / cx;                            // one CTA per SM, one wave
    if (slabs > (tokens + kS2Tok - 1) / kS2Tok) slabs = (tokens + kS2Tok - 1) / kS2Tok;
    long long per = (tokens + slabs - 1) / slabs;
    per = (per + kS2Tok - 1) / kS2Tok * kS2Tok;
    slabs = (tokens + per - 1) / per;
    if (slabs > 65535) return MONARCH_ERR_UNSUPPORTED;
    rect_dl_stream_kernel<<<dim3((unsigned)cx, (unsigned)slabs), kS2Threads, smem, s>>>(tm_dy, tm_u, dL, status, tokens, q,
                                                                                      b, r, (int)per);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

// dR on the tensor cores: bf16, b a multiple of 128 (the 128 TMEM lanes), b1 a multiple of 64
bool rect_wgrad_R_tc_available(int q, int b1, int b, int dtype)
{
    (void)q;
    return dtype == MONARCH_BF16 && b % 128 == 0 && b1 % 64 == 0;
}

int rect_wgrad_R_tc(const void *du, const void *x, float *dR, int64_t tokens, int q, int b1, int b, unsigned *status,
                    cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    if (b1 % 256 == 0) return tc::launch_wgrad<256>(du, x, dR, tokens, q, b1, b, status, s);
    return b1 % 128 == 0 ? tc::launch_wgrad<128>(du, x, dR, tokens, q, b1, b, status, s)
                         : tc::launch_wgrad<64>(du, x, dR, tokens, q, b1, b, status, s);
}

// adjoint of stage 1 on the tensor cores: dx[t][k*b1 + i] = sum_j R[k][j][i] du[t][k*b + j]
int rect_stage1_adjoint_tc(const void *du, const void *R, void *dx, int64_t tokens, int q, int b1, int b,
                           unsigned *status, cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    if (b1 % 256 == 0 && tokens > 128) {
        bool used = false;
        MONARCH_TRY(tc::launch_pair<true>(du, R, dx, tokens, q, b, b1, status, s, &used));
        if (used) return MONARCH_OK;
    }
    if (b1 % 256 == 0) return tc::launch<256, true>(du, R, dx, tokens, q, b, b1, status, s);
    return b1 % 128 == 0 ? tc::launch<128, true>(du, R, dx, tokens, q, b, b1, status, s)
                         : tc::launch<64, true>(du, R, dx, tokens, q, b, b1, status, s);
}

}  // namespace monarch
