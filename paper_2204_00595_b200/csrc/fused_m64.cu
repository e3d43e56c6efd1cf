// Fused Monarch forward for m = 64 (n = 4096), bf16 in/out, fp32 accumulation in TMEM.
//
// One persistent launch runs both block-diagonal stages and both permutations.  The work is
// cut into items that a CTA (one per SM) processes in a fixed interleaved order:
//
//   S1 item (128 tokens, 8 consecutive blocks k of R):
//       TMA brings x[128 x 64] and R_k[64 x 64] per block into 128B-swizzled K-major tiles;
//       tcgen05.mma (M=128 tokens, N=64, K=16) accumulates u[t][k][:] in TMEM columns
//       [64*kb, 64*kb+64).  With all 8 accumulators resident, the thread that owns token t picks
//       entry j of each block - a register renaming - and writes the 16 bytes
//       u'[t][j][8g..8g+8) into an L2-resident exchange buffer whose layout,
//       [64-token tile][j][k/8][t%64][k%8], makes that store fully coalesced (a warp writes 512
//       contiguous bytes) and is at the same time the canonical no-swizzle K-major operand
//       layout of stage 2: the inner permutation P^T costs no data movement at all.
//   S2 item (64 tokens, 16 consecutive blocks j of L):
//       one 8 KB bulk copy per block fetches u'_j[64 x 64] from L2, TMA fetches L_j;
//       tcgen05.mma (M=64, N=64) accumulates w[t][j][:]; the 16 accumulators sit in the two
//       16-lane halves of each TMEM sub-partition, so lanes i and i+16 of a warp hold blocks
//       j0..j0+7 and j0+8..j0+15 of the same token and together store the 32 contiguous bytes
//       y[t][l*64 + 16h .. 16h+16) - whole 32-byte sectors, which is what HBM writes need.
//
// S2 items of a token tile come `lag` tiles after its S1 items in the schedule and wait (with
// a bound) on a per-tile counter that S1 epilogues bump after their stores, so u' is consumed
// from L2 shortly after it is produced.  Warps: 0-3 drain TMEM, 4 issues TMA/bulk loads,
// 5 issues MMAs; an 8-slot shared-memory ring decouples loads from MMAs across items.
#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

constexpr int kM = 64;
constexpr int kN = kM * kM;
constexpr int kSlots = 8;
constexpr int kSlotBytes = 24576;            // 16 KB A + 8 KB B
constexpr int kSlotB = 16384;                // offset of B inside a slot
constexpr int kThreads = 192;
constexpr int kSmemBytes = kSlots * kSlotBytes + 1024;
constexpr unsigned kS1Arrivals = 8 * 4;      // 8 S1 items x 4 epilogue warps per 128-token tile
constexpr unsigned kS2Items = 8;             // S2 items per 128-token tile

struct FwdParams {
    __nv_bfloat16 *u;          // exchange buffer, [tiles64][64 j][8][64 t][8] bf16
    __nv_bfloat16 *y;
    unsigned *counters;        // one per 128-token tile, zero between calls
    unsigned *status;
    long long tokens;
    int tiles;                 // 128-token tiles
    int mode;                  // 0: S1 items only, 1: S2 items only, 2: both, dependency-tracked
    int lag;                   // tiles between a tile's S1 and S2 items (mode 2)
};

struct Item {
    int kind;   // 0 = S1, 1 = S2, -1 = none
    int tile;   // 128-token tile
    int sub;    // S1: block group g (0..7); S2: half*4 + h
};

// position in the global item order -> item.  Mode 2 order by tile step u: the 8 S1 items of
// tile u (while u < tiles), then the 8 S2 items of tile u - lag (once u >= lag).
__device__ __forceinline__ Item item_at(const FwdParams &p, long long pos)
{
    Item it = {-1, 0, 0};
    if (p.mode == 0 || p.mode == 1) {
        if (pos < (long long)p.tiles * 8) { it.kind = p.mode; it.tile = (int)(pos >> 3); it.sub = (int)(pos & 7); }
        return it;
    }
    const long long lag = p.lag < p.tiles ? p.lag : p.tiles;
    const long long a = lag * 8;                          // S1-only prefix
    const long long b = a + (p.tiles - lag) * 16;         // mixed region
    const long long c = b + lag * 8;                      // S2-only suffix
    if (pos < a) { it.kind = 0; it.tile = (int)(pos >> 3); it.sub = (int)(pos & 7); }
    else if (pos < b) {
        const long long q = pos - a;
        const int step = (int)(q >> 4), r = (int)(q & 15);
        if (r < 8) { it.kind = 0; it.tile = (int)lag + step; it.sub = r; }
        else { it.kind = 1; it.tile = step; it.sub = r - 8; }
    } else if (pos < c) {
        const long long q = pos - b;
        it.kind = 1; it.tile = (int)(p.tiles - lag + (q >> 3)); it.sub = (int)(q & 7);
    }
    return it;
}

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

__global__ void __launch_bounds__(kThreads, 1)
fused_fwd_m64_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_R,
                     const __grid_constant__ CUtensorMap tm_L, const FwdParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kSlots], bar_empty[kSlots], bar_acc_full, bar_acc_empty;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead;

    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc_full), 1);
        mbar_init(smem_u32(&bar_acc_empty), 4);
        fence_mbar_init();
        dead = 0;
        tma_prefetch_desc(&tm_x);
        tma_prefetch_desc(&tm_R);
        tma_prefetch_desc(&tm_L);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    const long long stride = gridDim.x;

    if (warp == 4) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t cnt = 0;
            bool ok = true;
            for (long long pos = blockIdx.x; ok; pos += stride) {
                const Item it = item_at(p, pos);
                if (it.kind < 0) break;
                if (it.kind == 1 && p.mode == 2) {
                    // wait until all S1 items of this tile have published their part of u'
                    const unsigned *ctr = p.counters + it.tile;
                    const unsigned long long t0 = global_timer_ns();
                    while (ld_acquire(ctr) < kS1Arrivals) {
                        if (*(volatile int *)&dead || global_timer_ns() - t0 > kWaitLimitNs) {
                            dead = 1;
                            atomicCAS(p.status, 0u, (unsigned)kErrPeerWait);
                            ok = false;
                            break;
                        }
                    }
                    if (!ok) break;
                    fence_proxy_async_global();
                }
                const int nblk = it.kind == 0 ? 8 : 16;
                for (int b = 0; b < nblk; ++b, ++cnt) {
                    const int s = cnt % kSlots;
                    if (!mbar_wait(smem_u32(&bar_empty[s]), ((cnt / kSlots) & 1) ^ 1, p.status, &dead,
                                   kErrSlotWait)) { ok = false; break; }
                    const uint32_t a = smem0 + s * kSlotBytes, w = a + kSlotB;
                    const uint32_t full = smem_u32(&bar_full[s]);
                    if (it.kind == 0) {
                        const int k = it.sub * 8 + b;
                        mbar_expect_tx(full, 16384 + 8192);
                        tma_load_2d(a, &tm_x, k * kM, it.tile * 128, full);
                        tma_load_2d(w, &tm_R, 0, k * kM, full);
                    } else {
                        const int half = it.sub >> 2, h = it.sub & 3;
                        const int j = h * 16 + b;
                        const long long tile64 = (long long)it.tile * 2 + half;
                        mbar_expect_tx(full, 8192 + 8192);
                        bulk_load(a, p.u + (tile64 * 64 + j) * 4096, 8192, full);
                        tma_load_2d(w, &tm_L, 0, j * kM, full);
                    }
                }
                if (ok && it.kind == 1 && p.mode == 2) {
                    // the last S2 item of a tile to get here clears the tile's counter for the next call
                    const unsigned old = atomicAdd(p.counters + it.tile, 1u);
                    if (old + 1 == kS1Arrivals + kS2Items) atomicExch(p.counters + it.tile, 0u);
                }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc1 = make_idesc_bf16(128, 64, 0, 0);
            constexpr uint32_t idesc2 = make_idesc_bf16(64, 64, 0, 0);
            uint32_t cnt = 0, nitem = 0;
            bool ok = true;
            for (long long pos = blockIdx.x; ok; pos += stride, ++nitem) {
                const Item it = item_at(p, pos);
                if (it.kind < 0) break;
                if (!mbar_wait(smem_u32(&bar_acc_empty), (nitem & 1) ^ 1, p.status, &dead, kErrTmemWait)) break;
                tc_fence_after();
                const int nblk = it.kind == 0 ? 8 : 16;
                for (int b = 0; b < nblk; ++b, ++cnt) {
                    const int s = cnt % kSlots;
                    if (!mbar_wait(smem_u32(&bar_full[s]), (cnt / kSlots) & 1, p.status, &dead, kErrTmaWait)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a = smem0 + s * kSlotBytes, w = a + kSlotB;
                    if (it.kind == 0) {
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            mma_f16_ss(tmem_base + b * 64, make_smem_desc(a + ks * 32, 16, 1024, kSwizzle128),
                                       make_smem_desc(w + ks * 32, 16, 1024, kSwizzle128), idesc1, ks != 0);
                    } else {
                        // accumulators 0-7 in lanes [0,16) of each sub-partition, 8-15 in lanes [16,32)
                        const uint32_t d = tmem_base + ((uint32_t)((b >> 3) * 16) << 16) + (b & 7) * 64;
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            mma_f16_ss(d, make_smem_desc(a + ks * 2048, 1024, 128, 0),
                                       make_smem_desc(w + ks * 32, 16, 1024, kSwizzle128), idesc2, ks != 0);
                    }
                    mma_commit(smem_u32(&bar_empty[s]));
                }
                if (ok) mma_commit(smem_u32(&bar_acc_full));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 0-3)
        const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
        uint32_t nitem = 0;
        for (long long pos = blockIdx.x;; pos += stride, ++nitem) {
            const Item it = item_at(p, pos);
            if (it.kind < 0) break;
            if (!mbar_wait(smem_u32(&bar_acc_full), nitem & 1, p.status, &dead, kErrMmaWait)) break;
            tc_fence_after();
            if (it.kind == 0) {
                const int r = warp * 32 + lane;
                const long long tile64 = (long long)it.tile * 2 + (r >> 6);
                uint8_t *dst = reinterpret_cast<uint8_t *>(p.u) + (tile64 * 64) * 8192 + it.sub * 1024 + (r & 63) * 16;
#pragma unroll 1
                for (int jc = 0; jc < 8; ++jc) {
                    uint32_t v[8][8];
#pragma unroll
                    for (int kb = 0; kb < 8; ++kb) tmem_ld8(lane_base + kb * 64 + jc * 8, v[kb]);
                    tmem_ld_wait();
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(v[0][q]), __uint_as_float(v[1][q]));
                        o.y = pack_bf16(__uint_as_float(v[2][q]), __uint_as_float(v[3][q]));
                        o.z = pack_bf16(__uint_as_float(v[4][q]), __uint_as_float(v[5][q]));
                        o.w = pack_bf16(__uint_as_float(v[6][q]), __uint_as_float(v[7][q]));
                        *reinterpret_cast<uint4 *>(dst + (size_t)(jc * 8 + q) * 8192) = o;
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty));
                if (p.mode == 2) {
                    // publish: the stores above must be visible to other SMs' bulk copies
                    fence_proxy_async_global();
                    __threadfence();
                    __syncwarp();
                    if (lane == 0) atomicAdd(p.counters + it.tile, 1u);
                }
            } else {
                const int half = it.sub >> 2, h = it.sub & 3;
                const long long t = (long long)it.tile * 128 + half * 64 + warp * 16 + (lane & 15);
                uint8_t *dst = reinterpret_cast<uint8_t *>(p.y) + (size_t)t * (kN * 2) + h * 32 + (lane >> 4) * 16;
                const bool live = t < p.tokens;
#pragma unroll 1
                for (int lc = 0; lc < 8; ++lc) {
                    uint32_t v[8][8];
#pragma unroll
                    for (int a = 0; a < 8; ++a) tmem_ld8(lane_base + a * 64 + lc * 8, v[a]);
                    tmem_ld_wait();
                    if (live) {
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            uint4 o;
                            o.x = pack_bf16(__uint_as_float(v[0][q]), __uint_as_float(v[1][q]));
                            o.y = pack_bf16(__uint_as_float(v[2][q]), __uint_as_float(v[3][q]));
                            o.z = pack_bf16(__uint_as_float(v[4][q]), __uint_as_float(v[5][q]));
                            o.w = pack_bf16(__uint_as_float(v[6][q]), __uint_as_float(v[7][q]));
                            *reinterpret_cast<uint4 *>(dst + (lc * 8 + q) * 128) = o;
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bar_acc_empty));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }

}  // namespace
}  // namespace tc

// Workspace: [status 256 B][tile counters, 64 KB][u' exchange buffer, tokens rounded up to 128].
constexpr size_t kFusedCounterBytes = 65536;

size_t fused_fwd_m64_workspace_bytes(int64_t tokens)
{
    const size_t tiles = (size_t)((tokens + 127) / 128);
    return MONARCH_STATUS_BYTES + kFusedCounterBytes + tc::align256(tiles * 128 * (size_t)tc::kN * 2);
}

int fused_fwd_m64(const void *x, const void *L, const void *R, void *y, int64_t tokens, void *ws,
                  int mode, cudaStream_t s)
{
    using namespace tc;
    if (tokens == 0) return MONARCH_OK;
    const long long tiles = (tokens + 127) / 128;
    if (tiles * 4 > (long long)kFusedCounterBytes) return MONARCH_ERR_UNSUPPORTED;
    CUtensorMap tm_x, tm_R, tm_L;
    MONARCH_TRY(encode_tmap_2d(&tm_x, x, (uint64_t)tokens, kN, kN * 2, 128, 64, 128));
    MONARCH_TRY(encode_tmap_2d(&tm_R, R, kN, kM, kM * 2, 64, 64, 128));
    MONARCH_TRY(encode_tmap_2d(&tm_L, L, kN, kM, kM * 2, 64, 64, 128));
    FwdParams p;
    p.status = (unsigned *)ws;
    p.counters = (unsigned *)((char *)ws + MONARCH_STATUS_BYTES);
    p.u = (__nv_bfloat16 *)((char *)ws + MONARCH_STATUS_BYTES + kFusedCounterBytes);
    p.y = (__nv_bfloat16 *)y;
    p.tokens = tokens;
    p.tiles = (int)tiles;
    p.lag = 24;
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        MONARCH_CUDA_TRY(cudaGetDevice(&dev));
        MONARCH_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        MONARCH_CUDA_TRY(cudaFuncSetAttribute(fused_fwd_m64_kernel,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    }
    auto launch = [&](int m) -> int {
        p.mode = m;
        const long long items = m == 2 ? tiles * 16 : tiles * 8;
        const unsigned grid = (unsigned)(items < sms ? items : sms);
        fused_fwd_m64_kernel<<<grid, kThreads, kSmemBytes, s>>>(tm_x, tm_R, tm_L, p);
        note_launch();
        MONARCH_CUDA_TRY(cudaGetLastError());
        return MONARCH_OK;
    };
    if (mode == 2) return launch(2);
    MONARCH_TRY(launch(0));
    return launch(1);
}

}  // namespace monarch
