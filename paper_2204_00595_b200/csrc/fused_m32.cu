// Fused forward y = P L P^T R x for m = 32 (n = 1024), bf16: both stages and both permutations inside one CTA.
//
// At this size a 64-token tile of the intermediate u' = P R x is 128 KB and fits the shared memory of one SM, so
// nothing is exchanged between SMs (Section 3.3 steps 1-3 with the permutations done on chip, as the method
// is meant to run): a persistent CTA per SM takes whole tiles.
//   stage 1: x arrives as 64 x 64 TMA boxes (two blocks k side by side, 128B swizzle), R_k pairs as 64 x 32 boxes;
//            M = 64, N = 32 MMAs accumulate 16 blocks at a time into one 16-lane half of TMEM (a "plane" of 512
//            columns; the two halves of a stage go to the two planes); the epilogue packs 8 blocks' results for one (t, j) into 16 bytes and writes them into
//            the shared-memory buffer U[j][k/8][t][k%8] - the P^T of step 2 is which columns are packed together,
//            and U[j] is, as it lies, the K-major A operand of stage 2.
//   stage 2: A = U[j], B = L_j (streamed as pairs), again 16 blocks j per plane;
//            the epilogue packs 16 blocks into the 32 bytes y[t][l*32 + 16s .. +16) (the final P), staged and
//            stored with 3-D TMA boxes.
// One thread issues all MMAs in the order S1a S1b S2a S2b per tile (a = blocks 0-15, b = 16-31); stage 1 of
// the next tile is issued straight after S2b of the current one and cannot complete before it (the tensor
// pipe is in order), so a single U buffer suffices.  The weights (64 KB + 64 KB) are re-streamed from L2 for
// every tile: there is no room to keep them next to U.
#include <cstdlib>

#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

constexpr int kM = 32;
constexpr int kN = kM * kM;
// warps: 0-7 epilogue (two halves of four), 8-9 loaders of (x, R) pairs, 10 loader of L pairs, 11 MMA,
// 12-13 store threads
constexpr int kEpiWarps = 8, kXWarp0 = 8, kLWarp = 10, kMmaWarp = 11, kStoreWarp0 = 12;
constexpr int kThreads = 14 * 32;
constexpr int kUBytes = 32 * 4096;                       // U[j][k/8 4][t 64][16 B]
constexpr int kXSlotBytes = 8192 + 4096, kXSlots = 4;    // x pair tile + R pair tile
constexpr int kLSlotBytes = 4096, kLSlots = 4;           // L pair tile
constexpr int kStageBytes = 8192, kStagesPerHalf = 2;
constexpr int kSmemBytes = kUBytes + kXSlots * kXSlotBytes + kLSlots * kLSlotBytes + 2 * kStagesPerHalf * kStageBytes + 1024;

struct P32 {
    unsigned *status;
    int tiles;
    long long *trace;            // optional per-CTA timeline (debug builds), else null
};

#ifdef MONARCH_TRACE
#define T32(item, slot, val) do { if (p.trace && (item) < 16) p.trace[((size_t)blockIdx.x * 16 + (item)) * 8 + (slot)] = (val); } while (0)
#define C32() clock64()
#else
#define T32(item, slot, val) do { } while (0)
#define C32() 0ll
#endif

struct Bars {
    uint64_t xfull[2], xempty[2];                     // ring slots are handed over in groups of two
    uint64_t lfull[2], lempty[2];
    uint64_t pl_full[2], pl_empty[2];                 // the two accumulator planes (16-lane halves of TMEM)
    uint64_t st_full[2 * kStagesPerHalf], st_free[2 * kStagesPerHalf];
};

__device__ __forceinline__ bool wait_fast(uint32_t bar, uint32_t parity, unsigned *status, volatile int *dead,
                                          unsigned code)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait(bar, parity, status, dead, code);
}

__global__ void __launch_bounds__(kThreads, 1)
fused_fwd_m32_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_R,
                     const __grid_constant__ CUtensorMap tm_L, const __grid_constant__ CUtensorMap tm_y, const P32 p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) Bars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead_s;

    const uint32_t U0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t xring0 = U0 + kUBytes;
    const uint32_t lring0 = xring0 + kXSlots * kXSlotBytes;
    const uint32_t stage0 = lring0 + kLSlots * kLSlotBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *dead = &dead_s;

    if (threadIdx.x == 0) {
        for (int g = 0; g < 2; ++g) {
            mbar_init(smem_u32(&bars.xfull[g]), 2);          // one (x, R) pair from each of the two loaders
            mbar_init(smem_u32(&bars.xempty[g]), 1);
            mbar_init(smem_u32(&bars.lfull[g]), 1);
            mbar_init(smem_u32(&bars.lempty[g]), 1);
        }
        for (int h = 0; h < 2; ++h) {
            mbar_init(smem_u32(&bars.pl_full[h]), 1);
            mbar_init(smem_u32(&bars.pl_empty[h]), kEpiWarps);
        }
        for (int k = 0; k < 2 * kStagesPerHalf; ++k) {
            mbar_init(smem_u32(&bars.st_full[k]), 4);
            mbar_init(smem_u32(&bars.st_free[k]), 1);
        }
        fence_mbar_init();
        dead_s = 0;
        tma_prefetch_desc(&tm_x); tma_prefetch_desc(&tm_R); tma_prefetch_desc(&tm_L); tma_prefetch_desc(&tm_y);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    const int first = (int)blockIdx.x, step = (int)gridDim.x;
    const uint32_t xf0 = smem_u32(bars.xfull), xe0 = smem_u32(bars.xempty);
    const uint32_t lf0 = smem_u32(bars.lfull), le0 = smem_u32(bars.lempty);
    const uint32_t plf0 = smem_u32(bars.pl_full), ple0 = smem_u32(bars.pl_empty);

    if (first >= p.tiles) {
        // nothing to do
    } else if (warp >= kXWarp0 && warp < kXWarp0 + 2) {
        // ------------------------------------------------------------ (x, R) loaders: warp pw takes pairs pw, pw+2, ...
        if (lane == 0) {
            const int pw = warp - kXWarp0;
            uint32_t ng = 0;                               // group use count: pairs (2 ng, 2 ng + 1) of the stream
            for (int tile = first; tile < p.tiles; tile += step) {
                bool ok = true;
#pragma unroll 1
                for (int G = 0; G < 8; ++G, ++ng) {
                    const uint32_t g = ng & 1, ph = (ng >> 1) & 1;
                    const int pr = G * 2 + pw;
                    if (!wait_fast(xe0 + g * 8, ph ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
                    const uint32_t dst = xring0 + (g * 2 + pw) * kXSlotBytes, full = xf0 + g * 8;
                    mbar_expect_tx(full, kXSlotBytes);
                    tma_load_2d(dst, &tm_x, pr * 64, tile * 64, full);            // blocks 2pr, 2pr+1: 64 columns
                    tma_load_2d(dst + 8192, &tm_R, 0, pr * 64, full);             // R rows of both blocks
                }
                if (!ok) break;
            }
        }
    } else if (warp == kLWarp) {
        // ------------------------------------------------------------ L loader
        if (lane == 0) {
            uint32_t ng = 0;
            for (int tile = first; tile < p.tiles; tile += step) {
                bool ok = true;
#pragma unroll 1
                for (int G = 0; G < 8; ++G, ++ng) {
                    const uint32_t g = ng & 1, ph = (ng >> 1) & 1;
                    if (!wait_fast(le0 + g * 8, ph ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
                    mbar_expect_tx(lf0 + g * 8, 2 * kLSlotBytes);
                    tma_load_2d(lring0 + (g * 2) * kLSlotBytes, &tm_L, 0, (G * 2) * 64, lf0 + g * 8);
                    tma_load_2d(lring0 + (g * 2 + 1) * kLSlotBytes, &tm_L, 0, (G * 2 + 1) * 64, lf0 + g * 8);
                }
                if (!ok) break;
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(64, 32, 0, 0);
            const uint64_t d_x = make_smem_desc(0, 16, 1024, kSwizzle128);   // x pair tile: 128-byte rows
            const uint64_t d_w = make_smem_desc(0, 16, 512, kSwizzle64);     // weight tiles: 64-byte rows
            const uint64_t d_u = make_smem_desc(0, 1024, 128, 0);            // U[j]: k chunks 1 KB apart
            // ring use counts; per plane: sub-items issued so far, completions of its `empty` barrier waited for
            uint32_t nx = 0, nl = 0, issued[2] = {0, 0}, c[2] = {0, 0};
            bool ok = true;
            // wait until the epilogue has drained `target` sub-items of plane P (completion n has parity n & 1)
            auto drained = [&](int P, uint32_t target) {
                while (ok && c[P] < target) {
                    if (!wait_fast(ple0 + P * 8, c[P] & 1, p.status, dead, kErrTmemWait)) ok = false;
                    ++c[P];
                }
                tc_fence_after();
            };
            [[maybe_unused]] int ntile = -1;
            for (int tile = first; ok && tile < p.tiles; tile += step) {
                ++ntile;
                // sub-items S1a S1b S2a S2b alternate between the two planes, so a half never waits for the
                // epilogue of the half before it; only stage 2 waits - for all of U
#pragma unroll 1
                for (int q = 0; q < 4 && ok; ++q) {
                    const int P = q & 1, h = q & 1;
                    const uint32_t plane = tmem_base + ((uint32_t)(P * 16) << 16);
                    [[maybe_unused]] const long long t_a = C32();
                    if (q == 2) drained(1, issued[1]);     // S1b's epilogue: U is complete
                    drained(P, issued[P]);                 // this plane has been read out
                    if (!ok) break;
                    [[maybe_unused]] const long long t_b = C32();
                    [[maybe_unused]] long long wsum = 0;
                    if (q < 2) {
                        // four groups per half and two in the ring: group G sits in ring position G & 1
#pragma unroll
                        for (int G = 0; G < 4; ++G, ++nx) {
                            const uint32_t g = G & 1, ph = (nx >> 1) & 1;
                            [[maybe_unused]] const long long w0 = C32();
                            if (!wait_fast(xf0 + g * 8, ph, p.status, dead, kErrTmaWait)) { ok = false; break; }
                            tc_fence_after();
                            wsum += C32() - w0;
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const uint32_t slot = xring0 + (g * 2 + e) * kXSlotBytes;
                                const uint64_t ax = d_x | (uint64_t)(slot >> 4);
                                const uint64_t bw = d_w | (uint64_t)((slot + 8192) >> 4);
#pragma unroll
                                for (int i = 0; i < 2; ++i) {
                                    const uint32_t d = plane + ((G * 2 + e) * 2 + i) * 32;
                                    // block 2pr+i: columns [32 i, +32) of the pair tile, rows [32 i, +32) of the R pair
                                    mma_f16_ss(d, ax + i * 4, bw + i * 128, idesc, 0);
                                    mma_f16_ss(d, ax + i * 4 + 2, bw + i * 128 + 2, idesc, 1);
                                }
                            }
                            mma_commit(xe0 + g * 8);
                        }
                    } else {
#pragma unroll
                        for (int G = 0; G < 4; ++G, ++nl) {
                            const uint32_t g = G & 1, ph = (nl >> 1) & 1;
                            [[maybe_unused]] const long long w0 = C32();
                            if (!wait_fast(lf0 + g * 8, ph, p.status, dead, kErrTmaWait)) { ok = false; break; }
                            tc_fence_after();
                            wsum += C32() - w0;
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const uint64_t bl = d_w | (uint64_t)((lring0 + (g * 2 + e) * kLSlotBytes) >> 4);
#pragma unroll
                                for (int i = 0; i < 2; ++i) {
                                    const int jb = (G * 2 + e) * 2 + i;
                                    const uint32_t d = plane + jb * 32;
                                    const uint64_t au = d_u | (uint64_t)((U0 + (h * 16 + jb) * 4096) >> 4);
                                    mma_f16_ss(d, au, bl + i * 128, idesc, 0);
                                    mma_f16_ss(d, au + 128, bl + i * 128 + 2, idesc, 1);
                                }
                            }
                            mma_commit(le0 + g * 8);
                        }
                    }
                    if (!ok) break;
                    mma_commit(plf0 + P * 8);
                    T32(ntile * 4 + q, 0, t_a); T32(ntile * 4 + q, 1, t_b - t_a); T32(ntile * 4 + q, 2, wsum);
                    T32(ntile * 4 + q, 3, C32());
                    ++issued[P];
                }
            }
        }
    } else if (warp < kEpiWarps) {
        // ------------------------------------------------------------ epilogues
        const int q4 = warp & 3, sub = warp >> 2, hl = lane >> 4;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q4 * 32) << 16);
        const int row = q4 * 16 + (lane & 15);
        const uint32_t my_stage = stage0 + sub * kStagesPerHalf * kStageBytes;
        const uint32_t stf0 = smem_u32(bars.st_full) + sub * kStagesPerHalf * 8;
        const uint32_t stfree0 = smem_u32(bars.st_free) + sub * kStagesPerHalf * 8;
        uint32_t np[2] = {0, 0}, nchunk = 0;          // sub-items seen per plane
        bool ok = true;
        for (int tile = first; ok && tile < p.tiles; tile += step) {
            // ---- stage 1 halves: half h sits in plane h (lanes 16 h .. 16 h + 15 of every quarter) -> U
#pragma unroll 1
            for (int h = 0; h < 2 && ok; ++h) {
                if (!wait_fast(plf0 + h * 8, np[h] & 1, p.status, dead, kErrMmaWait)) { ok = false; break; }
                ++np[h];
                tc_fence_after();
                // this warp: rows j in [16 sub, 16 sub + 16), in two chunks of 8; blocks k of this half in two
                // groups of 8 -> U chunk index 2h + g
#pragma unroll 1
                for (int jc = 0; jc < 2; ++jc) {
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        uint32_t v[8][8];
#pragma unroll
                        for (int kb = 0; kb < 8; ++kb) tmem_ld8(lane_base + (g * 8 + kb) * 32 + sub * 16 + jc * 8, v[kb]);
                        tmem_ld_wait();
                        if (hl == h) {
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                const uint32_t o0 = pack_bf16(__uint_as_float(v[0][q]), __uint_as_float(v[1][q]));
                                const uint32_t o1 = pack_bf16(__uint_as_float(v[2][q]), __uint_as_float(v[3][q]));
                                const uint32_t o2 = pack_bf16(__uint_as_float(v[4][q]), __uint_as_float(v[5][q]));
                                const uint32_t o3 = pack_bf16(__uint_as_float(v[6][q]), __uint_as_float(v[7][q]));
                                const int j = sub * 16 + jc * 8 + q;
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(U0 + j * 4096 + (h * 2 + g) * 1024 + row * 16),
                                             "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                            }
                        }
                    }
                }
                tc_fence_before();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(ple0 + h * 8);
            }
            // ---- stage 2 halves: half h in plane h -> y
#pragma unroll 1
            for (int h = 0; h < 2 && ok; ++h) {
                if (!wait_fast(plf0 + h * 8, np[h] & 1, p.status, dead, kErrMmaWait)) { ok = false; break; }
                ++np[h];
                tc_fence_after();
#pragma unroll 1
                for (int c = sub; c < 8; c += 2, ++nchunk) {
                    const uint32_t k = nchunk & (kStagesPerHalf - 1);
                    const uint32_t sbuf = my_stage + k * kStageBytes;
                    if (!wait_fast(stfree0 + k * 8, ((nchunk / kStagesPerHalf) & 1) ^ 1, p.status, dead, kErrSlotWait)) { ok = false; break; }
                    // chunk = 4 consecutive output rows l; 16 blocks j of this half -> 32 bytes per (l, t)
                    uint32_t v[16][4];
#pragma unroll
                    for (int a = 0; a < 16; ++a) tmem_ld4(lane_base + a * 32 + c * 4, v[a]);
                    tmem_ld_wait();
                    if (hl == h) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const uint32_t o0 = pack_bf16(__uint_as_float(v[e * 8 + 0][q]), __uint_as_float(v[e * 8 + 1][q]));
                                const uint32_t o1 = pack_bf16(__uint_as_float(v[e * 8 + 2][q]), __uint_as_float(v[e * 8 + 3][q]));
                                const uint32_t o2 = pack_bf16(__uint_as_float(v[e * 8 + 4][q]), __uint_as_float(v[e * 8 + 5][q]));
                                const uint32_t o3 = pack_bf16(__uint_as_float(v[e * 8 + 6][q]), __uint_as_float(v[e * 8 + 7][q]));
                                // staging [l local 4][t 64][16 j]
                                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sbuf + q * 2048 + row * 32 + e * 16),
                                             "r"(o0), "r"(o1), "r"(o2), "r"(o3) : "memory");
                            }
                        }
                    }
                    if (c + 2 >= 8) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(ple0 + h * 8);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(stf0 + k * 8);
                }
            }
        }
    } else if (warp >= kStoreWarp0 && warp < kStoreWarp0 + 2) {
        // ------------------------------------------------------------ store threads (one per epilogue half)
        if (lane == 0) {
            const int sub = warp - kStoreWarp0;
            const uint32_t my_stage = stage0 + sub * kStagesPerHalf * kStageBytes;
            const uint32_t stf0 = smem_u32(bars.st_full) + sub * kStagesPerHalf * 8;
            const uint32_t stfree0 = smem_u32(bars.st_free) + sub * kStagesPerHalf * 8;
            uint32_t nchunk = 0;
            int unfreed = -1;
            bool ok = true;
            for (int tile = first; ok && tile < p.tiles; tile += step) {
#pragma unroll 1
                for (int h = 0; h < 2 && ok; ++h) {
#pragma unroll 1
                    for (int c = sub; c < 8; c += 2, ++nchunk) {
                        const uint32_t k = nchunk & (kStagesPerHalf - 1);
                        if (!wait_fast(stf0 + k * 8, (nchunk / kStagesPerHalf) & 1, p.status, dead, kErrMmaWait)) { ok = false; break; }
                        // y as [l][t][j]: box 16 j x 64 t x 4 l; rows past the last token are clipped
                        asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(&tm_y),
                                     "r"(my_stage + k * kStageBytes), "r"(h * 16), "r"(tile * 64), "r"(c * 4) : "memory");
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

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

}  // namespace
}  // namespace tc

// Workspace: only the status word is used.
int fused_fwd_m32(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws, cudaStream_t s)
{
    using namespace tc;
    if (tokens == 0) return MONARCH_OK;
    const long long tiles = (tokens + 63) / 64;
    if (tiles > 0x7fffffffLL / 64) return MONARCH_ERR_UNSUPPORTED;
    CUtensorMap tm_x, tm_R, tm_L, tm_y;
    MONARCH_TRY(encode_tmap_2d(&tm_x, x, (uint64_t)tokens, kN, kN * 2, 64, 64, 128));     // two blocks per box
    MONARCH_TRY(encode_tmap_2d(&tm_R, R, kN, kM, kM * 2, 64, 32, 64));                     // two blocks per box
    MONARCH_TRY(encode_tmap_2d(&tm_L, L, kN, kM, kM * 2, 64, 32, 64));
    {
        // y as [l][t][j] bf16; a store moves 16 j x 64 t x 4 l
        const uint64_t ydims[3] = {32, (uint64_t)tokens, 32}, ystrides[2] = {(uint64_t)kN * 2, 64};
        const uint32_t ybox[3] = {16, 64, 4};
        MONARCH_TRY(encode_tmap_nd(&tm_y, y, 2, 3, ydims, ystrides, ybox));
    }
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(fused_fwd_m32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          kSmemBytes));
    P32 p;
    p.status = (unsigned *)ws;
    p.tiles = (int)tiles;
    p.trace = nullptr;
#ifdef MONARCH_TRACE
    if (const char *e = getenv("MONARCH_TRACE_PTR")) p.trace = (long long *)strtoull(e, nullptr, 0);
#endif
    const int grid = tiles < sms ? (int)tiles : sms;
    fused_fwd_m32_kernel<<<grid, kThreads, kSmemBytes, s>>>(tm_x, tm_R, tm_L, tm_y, p);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

}  // namespace monarch
