// Backward pass as a chain of tensor-core launches for the block sizes that have no fused kernel (bf16):
//     z  = P dy                          (stride permutation, a pure data movement)
//     du = P blockdiag(L^T) z            (one stage of tc_stage.cu with transposed blocks; natural du[t][k][j])
//     dx = blockdiag(R^T) du             (the same stage kernel without its output permutation)
//     u' = P blockdiag(R) x              (forward stage 1)
//     dR[k] = sum_t du_k^T x_k,  dL[j] = sum_t z_j^T u'_j      (token reductions on tcgen05, m = 128)
// These are the adjoints of Section 3.3 steps 1-3 written with G(W) = P blockdiag(W):
// M^T = R^T P L^T P = blockdiag(R^T) G(L^T) P.  Everything between two launches goes through the caller's
// workspace; this family trades HBM traffic for reach.
#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

// z[t][a*m + b] = v[t][b*m + a]: a transpose of every token's m x m view, 32 x 32 tiles through shared memory
__global__ void __launch_bounds__(256) permute_kernel(const __nv_bfloat16 *__restrict__ v, __nv_bfloat16 *__restrict__ z,
                                                      int m, long long tokens)
{
    __shared__ __nv_bfloat16 tile[32][34];
    const long long t = blockIdx.z;
    const int a0 = blockIdx.y * 32, b0 = blockIdx.x * 32;
    const __nv_bfloat16 *src = v + t * (long long)m * m;
    __nv_bfloat16 *dst = z + t * (long long)m * m;
    for (int r = threadIdx.y; r < 32; r += 8) tile[r][threadIdx.x] = src[(long long)(b0 + r) * m + a0 + threadIdx.x];
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += 8) dst[(long long)(a0 + r) * m + b0 + threadIdx.x] = tile[threadIdx.x][r];
}

// The same with 16-byte global accesses: one CTA per token; the m x m view goes to shared memory as it is stored
// (pitch m/2 + 1 words) and leaves as rows of the transpose, each thread gathering the 8 elements of one 16-byte piece.
__global__ void __launch_bounds__(256) permute_vec_kernel(const __nv_bfloat16 *__restrict__ v, __nv_bfloat16 *__restrict__ z,
                                                          int m)
{
    extern __shared__ uint32_t ptile[];                        // [m][m/2 + 1] words
    const int pitch = m / 2 + 1, chunks = m * m / 8, cpr = m / 8;
    const __nv_bfloat16 *src = v + (size_t)blockIdx.x * m * m;
    __nv_bfloat16 *dst = z + (size_t)blockIdx.x * m * m;
    for (int c = threadIdx.x; c < chunks; c += 256) {
        const int row = c / cpr, c8 = c % cpr;
        const uint4 q = *reinterpret_cast<const uint4 *>(src + (size_t)c * 8);
        uint32_t *d = ptile + row * pitch + c8 * 4;
        d[0] = q.x; d[1] = q.y; d[2] = q.z; d[3] = q.w;
    }
    __syncthreads();
    // a warp takes a patch of 8 output rows x 4 pieces: its loads of one source row hit 4 x 4 distinct banks, and
    // every output row gets 64 contiguous bytes
    const unsigned short *h = reinterpret_cast<const unsigned short *>(ptile);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int pcols = cpr / 4, patches = (m / 8) * pcols;
    for (int pidx = warp; pidx < patches; pidx += 8) {
        const int row = (pidx / pcols) * 8 + (lane >> 2), c8 = (pidx % pcols) * 4 + (lane & 3);   // output row = input column
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t lo = h[(size_t)(c8 * 8 + 2 * e) * pitch * 2 + row];
            const uint32_t hi = h[(size_t)(c8 * 8 + 2 * e + 1) * pitch * 2 + row];
            w[e] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4 *>(dst + ((size_t)row * cpr + c8) * 8) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// Wt[b][c][e] = W[b][e][c] for every block
__global__ void __launch_bounds__(256) transpose_blocks_kernel(const __nv_bfloat16 *__restrict__ W,
                                                               __nv_bfloat16 *__restrict__ Wt, int m)
{
    __shared__ __nv_bfloat16 tile[32][34];
    const int b = blockIdx.z;
    const int e0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    const __nv_bfloat16 *src = W + (long long)b * m * m;
    __nv_bfloat16 *dst = Wt + (long long)b * m * m;
    for (int r = threadIdx.y; r < 32; r += 8) tile[r][threadIdx.x] = src[(long long)(e0 + r) * m + c0 + threadIdx.x];
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += 8) dst[(long long)(c0 + r) * m + e0 + threadIdx.x] = tile[threadIdx.x][r];
}

// ---------------------------------------------------------------------------------------------- token reduction
// out[g][r][c] += sum_t A[t][g*m + r] * B[t][g*m + c] for m x m blocks, m = 32, 64 or 128 (dR from du and x, dL from
// P dy and u').  The kernel works on windows of 128 columns: D = A_w^T B_w (128 x 128, contraction over tokens) holds
// the sums of the window's 128 / m blocks on its diagonal; the off-diagonal part pairs different blocks and is
// dropped (the tensor pipe is idle anyway).  Both operands are read token-major (MN-major descriptors over 64-token x
// 64-column TMA boxes, 128B swizzle), a CTA owns 4 windows (4 accumulators of 128 lanes x 128 columns fill TMEM) and
// a slice of the token tiles, and adds its partial sums to the output with vector reductions in L2 at the end.
constexpr int kWM = 128;
constexpr int kWSlotBytes = 32768;             // A tile 16 KB + B tile 16 KB (two 64-column halves each)
constexpr int kWSlots = 6;
constexpr int kWSmem = kWSlots * kWSlotBytes + 1024;
constexpr int kWThreads = 6 * 32;              // warps 0-3 epilogue, 4 loader, 5 MMA

struct WgradParams {
    float *out;
    float *part;           // fixed summation order: slice y stores its sums to part[y][block][m][m] instead of adding them to out
    unsigned *status;
    int tiles, slices;
    int m;                 // block size: 128 (a window is one block), 64 or 32 (its 2 or 4 diagonal sub-blocks are blocks)
    int windows;           // 128-column windows of a token row (n / 128)
};

__device__ __forceinline__ bool wait_fast(uint32_t bar, uint32_t parity, unsigned *status, volatile int *dead,
                                          unsigned code)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait(bar, parity, status, dead, code);
}

__global__ void __launch_bounds__(kWThreads, 1)
tc_wgrad_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, const WgradParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kWSlots], bar_empty[kWSlots], bar_acc;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead;

    const uint32_t ring0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int blk0 = blockIdx.x * 4, first = blockIdx.y, step = p.slices;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kWSlots; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_acc), 1);
        fence_mbar_init();
        dead = 0;
        tma_prefetch_desc(&tm_a);
        tma_prefetch_desc(&tm_b);
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
        if (warp == 4) {
            if (lane == 0) {
                int slot = 0;
                uint32_t ph = 0;
                for (int tile = first; tile < p.tiles && !dead; tile += step) {
#pragma unroll 1
                    for (int b = 0; b < 4 && blk0 + b < p.windows; ++b) {
                        if (!wait_fast(empty0 + slot * 8, ph ^ 1, p.status, &dead, kErrSlotWait)) break;
                        const uint32_t dst = ring0 + slot * kWSlotBytes, full = full0 + slot * 8;
                        const int col = (blk0 + b) * kWM;
                        mbar_expect_tx(full, kWSlotBytes);
                        tma_load_2d(dst, &tm_a, col, tile * 64, full);
                        tma_load_2d(dst + 8192, &tm_a, col + 64, tile * 64, full);
                        tma_load_2d(dst + 16384, &tm_b, col, tile * 64, full);
                        tma_load_2d(dst + 24576, &tm_b, col + 64, tile * 64, full);
                        if (++slot == kWSlots) { slot = 0; ph ^= 1; }
                    }
                }
            }
        } else if (warp == 5) {
            if (lane == 0) {
                constexpr uint32_t idesc = make_idesc_bf16(128, 128, 1, 1);
                // two 64-column swizzle atoms 8 KB apart along M (N); 8-token groups 1 KB apart along K
                const uint64_t desc = make_smem_desc(0, 8192, 1024, kSwizzle128);
                int slot = 0;
                uint32_t ph = 0;
                bool ok = true;
                for (int tile = first; ok && tile < p.tiles; tile += step) {
                    const uint32_t accum = tile != first;
#pragma unroll 1
                    for (int b = 0; b < 4 && blk0 + b < p.windows; ++b) {
                        if (!wait_fast(full0 + slot * 8, ph, p.status, &dead, kErrTmaWait)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t ad = desc | (uint64_t)((ring0 + slot * kWSlotBytes) >> 4);
                        const uint64_t bd = ad + (16384 >> 4);
                        const uint32_t d = tmem_base + b * 128;
                        mma_f16_ss(d, ad, bd, idesc, accum);
                        mma_f16_ss(d, ad + 128, bd + 128, idesc, 1);          // 16 tokens = 2 KB further
                        mma_f16_ss(d, ad + 256, bd + 256, idesc, 1);
                        mma_f16_ss(d, ad + 384, bd + 384, idesc, 1);
                        mma_commit(empty0 + slot * 8);
                        if (++slot == kWSlots) { slot = 0; ph ^= 1; }
                    }
                }
                if (ok) mma_commit(acc);
            }
        } else if (warp < 4) {
            if (mbar_wait(acc, 0, p.status, &dead, kErrMmaWait)) {
                tc_fence_after();
                const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
                const int row = warp * 32 + lane;
#pragma unroll 1
                for (int b = 0; b < 4 && blk0 + b < p.windows; ++b) {
                    // the window's diagonal m x m sub-blocks are the blocks' sums (the rest of the 128 x 128 product pairs
                    // rows and columns of different blocks and is dropped); row `row` of the window is row g % m of block g / m
                    const int g = (blk0 + b) * kWM + row, c0 = (row / p.m) * p.m;     // c0 is uniform over a warp: m >= 32
                    float *out = (p.part ? p.part + (size_t)blockIdx.y * p.windows * kWM * p.m : p.out) +
                                 ((long long)(g / p.m) * p.m + g % p.m) * p.m - c0;
#pragma unroll 1
                    for (int c = c0; c < c0 + p.m; c += 16) {
                        uint32_t v[16];
                        tmem_ld16(lane_base + b * 128 + c, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if (p.part)
                                *reinterpret_cast<float4 *>(out + c + e * 4) =
                                    make_float4(__uint_as_float(v[e * 4]), __uint_as_float(v[e * 4 + 1]),
                                                __uint_as_float(v[e * 4 + 2]), __uint_as_float(v[e * 4 + 3]));
                            else
                                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(out + c + e * 4),
                                             "f"(__uint_as_float(v[e * 4])), "f"(__uint_as_float(v[e * 4 + 1])),
                                             "f"(__uint_as_float(v[e * 4 + 2])), "f"(__uint_as_float(v[e * 4 + 3]))
                                             : "memory");
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

// out[i] += part[0][i] + part[1][i] + ... in slice order, for the n*m elements of a weight gradient
__global__ void __launch_bounds__(256) add_slices_kernel(float *__restrict__ out, const float *__restrict__ part, int slices,
                                                         int elems)
{
    const int i = (blockIdx.x * 256 + threadIdx.x) * 4;
    if (i >= elems) return;
    float4 acc = *reinterpret_cast<const float4 *>(part + i);
    for (int s = 1; s < slices; ++s) {
        const float4 v = *reinterpret_cast<const float4 *>(part + (size_t)s * elems + i);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    float4 o = *reinterpret_cast<float4 *>(out + i);
    o.x += acc.x; o.y += acc.y; o.z += acc.z; o.w += acc.w;
    *reinterpret_cast<float4 *>(out + i) = o;
}

// slices of the token tiles that fit the scratch for one gradient's partial sums
int max_wgrad_slices(int m) { return (int)(kTcPartialBytes / 2 / ((size_t)m * m * m * sizeof(float))); }

// out[g][r][c] += sum_t A[t][g*m + r] B[t][g*m + c] for every block g (m = 32, 64 or 128; A, B token-major [tokens][m*m]).
// part != null (kTcPartialBytes / 2 of scratch): every slice of the tokens stores its sums there and a second launch adds
// them to out in slice order - the same bits on every run; else the slices add to out with reductions in L2.
int launch_wgrad(const void *A, const void *B, float *out, int64_t tokens, int m, unsigned *status, cudaStream_t s,
                 float *part = nullptr)
{
    if (tokens == 0) return MONARCH_OK;
    const int n = m * m;
    CUtensorMap tm_a, tm_b;
    MONARCH_TRY(encode_tmap_2d(&tm_a, A, (uint64_t)tokens, n, (uint64_t)n * 2, 64, 64, 128));
    MONARCH_TRY(encode_tmap_2d(&tm_b, B, (uint64_t)tokens, n, (uint64_t)n * 2, 64, 64, 128));
    // per call: the SM count and the shared-memory attribute belong to the current device, and a first-call
    // cache would not be safe against two host threads
    int sms = 0;
    MONARCH_TRY(current_device_sms(&sms));
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(tc_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kWSmem));
    WgradParams p;
    p.out = out;
    p.part = part;
    p.status = status;
    p.tiles = (int)((tokens + 63) / 64);
    p.m = m;
    p.windows = n / kWM;
    const int groups = (p.windows + 3) / 4;          // a CTA keeps the accumulators of four windows in TMEM
    int slices = sms / groups;
    if (slices < 1) slices = 1;
    if (slices > p.tiles) slices = p.tiles;
    if (part != nullptr && slices > max_wgrad_slices(m)) slices = max_wgrad_slices(m);
    p.slices = slices;
    tc_wgrad_kernel<<<dim3(groups, slices), kWThreads, kWSmem, s>>>(tm_a, tm_b, p);
    note_launch();
    if (part != nullptr) {
        const int elems = n * m;
        add_slices_kernel<<<(elems / 4 + 255) / 256, 256, 0, s>>>(out, part, slices, elems);
        note_launch();
    }
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

int permute(const void *v, void *z, int m, int64_t tokens, cudaStream_t s)
{
    if (tokens == 0) return MONARCH_OK;
    if (m % 32 == 0 && m <= 128 && tokens <= 0x7fffffffLL) {
        const int smem = m * (m / 2 + 1) * 4;
        permute_vec_kernel<<<(unsigned)tokens, 256, smem, s>>>((const __nv_bfloat16 *)v, (__nv_bfloat16 *)z, m);
        note_launch();
        MONARCH_CUDA_TRY(cudaGetLastError());
        return MONARCH_OK;
    }
    // grid.z carries the token index: at most 65535 per launch
    const __nv_bfloat16 *src = (const __nv_bfloat16 *)v;
    __nv_bfloat16 *dst = (__nv_bfloat16 *)z;
    for (int64_t t0 = 0; t0 < tokens; t0 += 65535) {
        const int64_t nt = tokens - t0 < 65535 ? tokens - t0 : 65535;
        permute_kernel<<<dim3(m / 32, m / 32, (unsigned)nt), dim3(32, 8), 0, s>>>(src + t0 * m * m, dst + t0 * m * m, m, nt);
        note_launch();
    }
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

int transpose_blocks(const void *W, void *Wt, int m, cudaStream_t s)
{
    transpose_blocks_kernel<<<dim3(m / 32, m / 32, m), dim3(32, 8), 0, s>>>((const __nv_bfloat16 *)W, (__nv_bfloat16 *)Wt, m);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }

struct Layout {
    char *z, *du, *u, *Lt, *Rt;
};
Layout carve(void *ws, int64_t tokens, int m)
{
    const size_t act = align256((size_t)tokens * m * m * 2), wb = align256((size_t)m * m * m * 2);
    Layout l;
    l.z = (char *)ws + MONARCH_STATUS_BYTES;
    l.du = l.z + act;
    l.u = l.du + act;
    l.Lt = l.u + act;
    l.Rt = l.Lt + wb;
    return l;
}

}  // namespace
}  // namespace tc

// Workspace: [status][z][du][u'][L^T][R^T]; m = 128 has its own layout (chain_m128.cu)
size_t tc_staged_bwd_workspace_bytes(int64_t tokens, int m, bool fixed_order)
{
    if (m == 128) return chain_bwd_m128_workspace_bytes(tokens);
    const size_t act = tc::align256((size_t)tokens * m * m * 2), wb = tc::align256((size_t)m * m * m * 2);
    return MONARCH_STATUS_BYTES + 3 * act + 2 * wb + (fixed_order ? kTcPartialBytes : 0);
}

// want_dx / want_dw select the outputs
int tc_staged_bwd(const void *x, const void *dy, const void *L, const void *R, void *dx, float *dL, float *dR,
                  int accumulate, int want_dx, int want_dw, int64_t tokens, int m, void *ws, cudaStream_t s,
                  const void *saved_up, bool fixed_order)
{
    using namespace tc;
    if (want_dw && m != 32 && m != 64 && m != 128) return MONARCH_ERR_UNSUPPORTED;
    if (m == 128) {
        // chain of block GEMMs on token-innermost intermediates (chain_m128.cu)
        if (tokens == 0 && want_dw && !accumulate) {
            const size_t gb = (size_t)m * m * m * sizeof(float);
            MONARCH_CUDA_TRY(cudaMemsetAsync(dL, 0, gb, s));
            MONARCH_CUDA_TRY(cudaMemsetAsync(dR, 0, gb, s));
        }
        return chain_bwd_m128(x, dy, L, R, saved_up, dx, dL, dR, accumulate, want_dx, want_dw, tokens, ws, s);
    }
    unsigned *status = (unsigned *)ws;
    const Layout l = carve(ws, tokens, m);
    if (want_dw && !accumulate) {
        const size_t gb = (size_t)m * m * m * sizeof(float);
        MONARCH_CUDA_TRY(cudaMemsetAsync(dL, 0, gb, s));
        MONARCH_CUDA_TRY(cudaMemsetAsync(dR, 0, gb, s));
    }
    if (tokens == 0) return MONARCH_OK;
    MONARCH_TRY(transpose_blocks(L, l.Lt, m, s));
    MONARCH_TRY(permute(dy, l.z, m, tokens, s));
    MONARCH_TRY(tc_stage(m, l.z, l.Lt, l.du, nullptr, 0, tokens, status, s));             // du[t][k][j]
    if (want_dx) {
        MONARCH_TRY(transpose_blocks(R, l.Rt, m, s));
        MONARCH_TRY(tc_stage(m, l.du, l.Rt, dx, nullptr, 0, tokens, status, s, 1));       // dx, no permutation
    }
    if (want_dw) {
        MONARCH_TRY(tc_stage(m, x, R, l.u, nullptr, 0, tokens, status, s));               // u'[t][j][k]
        // fixed summation order on request: the slices' sums go through the scratch behind R^T (one half per gradient)
        float *part = fixed_order ? (float *)(l.Rt + align256((size_t)m * m * m * 2)) : nullptr;
        MONARCH_TRY(launch_wgrad(l.du, x, dR, tokens, m, status, s, part));
        MONARCH_TRY(launch_wgrad(l.z, l.u, dL, tokens, m, status, s, part ? part + kTcPartialBytes / 2 / sizeof(float) : nullptr));
    }
    return MONARCH_OK;
}

}  // namespace monarch
