// One block-diagonal stage on the tcgen05 tensor cores (bf16 in, fp32 accumulate in TMEM):
//   out[t][e*m + b] = act( sum_c W[b][e][c] * in[t][b*m + c] + bias[e*m + b] )
// i.e. multiply every length-m segment of a token row by its block, then scatter with the
// stride permutation P (or, with `natural` set, leave the result in place: out[t][b*m + e]).  Two launches give the forward pass (M = (P L)(P R)), four the
// feed-forward block.  The intermediate goes through the caller's workspace, so this family
// is bounded by twice the HBM traffic of the fused kernels; it serves the sizes and calls
// that have no fused kernel.
//
// CTA = 128 tokens x 16 consecutive blocks x 32 output rows.  TMA brings each block's token
// tile [128 x m] and weight rows [NJ x m] into 128-byte (64-byte for m = 32) swizzled
// K-major tiles through a 4-slot ring; one thread issues the MMAs (M = 128 tokens, N = NJ,
// K = 16 per instruction), block b accumulating into TMEM columns [b*NJ, (b+1)*NJ).  With all
// sixteen accumulators resident, the thread that owns a token (a TMEM lane) picks element e of
// each of the 16 blocks - a register renaming, not a data movement - packs them to bf16 and
// writes the 32 contiguous bytes out[t][e*m + b0 .. b0+15].
#include "tc_common.cuh"

namespace monarch {
namespace tc {
namespace {

template <int M> struct StageCfg {
    static constexpr int KC = M < 64 ? M : 64;          // K elements per swizzled chunk
    static constexpr int NKC = M / KC;
    static constexpr int NJ = 32;                       // output rows per CTA
    static constexpr int NB = 16;                       // blocks per CTA: the permuted output leaves in 32-byte
                                                        // pieces (16-byte pieces reach only ~1 TB/s)
    static constexpr int TOK = 128;
    static constexpr int SWZ_BYTES = KC * 2;            // 64 or 128
    static constexpr uint32_t LAYOUT = SWZ_BYTES == 128 ? kSwizzle128 : kSwizzle64;
    static constexpr int A_CHUNK = TOK * KC * 2;
    static constexpr int B_CHUNK = NJ * KC * 2;
    static constexpr int A_BYTES = A_CHUNK * NKC;
    static constexpr int B_BYTES = B_CHUNK * NKC;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = 4;
    static constexpr int TMEM_COLS = NB * NJ;           // 512
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024;
    static_assert(A_BYTES % 1024 == 0 && B_BYTES % 1024 == 0, "swizzle atoms need 1 KB alignment");
};

template <int M>
__global__ void __launch_bounds__(128)
tc_stage_kernel(const __grid_constant__ CUtensorMap tm_in, const __grid_constant__ CUtensorMap tm_w,
                __nv_bfloat16 *__restrict__ out, const __nv_bfloat16 *__restrict__ bias, int gelu,
                int natural, long long tokens, unsigned *status)
{
    using C = StageCfg<M>;
    constexpr int n = M * M;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[C::STAGES], bar_empty[C::STAGES], bar_accum;
    __shared__ uint32_t tmem_base_s;
    __shared__ int dead;

    const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long t0 = (long long)blockIdx.x * C::TOK;
    const int b0 = blockIdx.y * C::NB;
    const int e0 = blockIdx.z * C::NJ;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);
        }
        mbar_init(smem_u32(&bar_accum), 1);
        fence_mbar_init();
        dead = 0;
        tma_prefetch_desc(&tm_in);
        tma_prefetch_desc(&tm_w);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_s), C::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    if (warp == 0 && lane == 0) {
        // producer: one slot per block
        for (int b = 0; b < C::NB; ++b) {
            const int s = b % C::STAGES;
            if (b >= C::STAGES &&
                !mbar_wait(smem_u32(&bar_empty[s]), ((b / C::STAGES) - 1) & 1, status, &dead, kErrSlotWait))
                break;
            const uint32_t a = smem0 + s * C::STAGE_BYTES, w = a + C::A_BYTES;
            const uint32_t full = smem_u32(&bar_full[s]);
            mbar_expect_tx(full, C::STAGE_BYTES);
#pragma unroll
            for (int kc = 0; kc < C::NKC; ++kc) {
                tma_load_2d(a + kc * C::A_CHUNK, &tm_in, (b0 + b) * M + kc * C::KC, (int)t0, full);
                tma_load_2d(w + kc * C::B_CHUNK, &tm_w, kc * C::KC, (b0 + b) * M + e0, full);
            }
        }
    } else if (warp == 1 && lane == 0) {
        // MMA issuer
        constexpr uint32_t idesc = make_idesc_bf16(C::TOK, C::NJ, 0, 0);
        bool ok = true;
        for (int b = 0; b < C::NB && ok; ++b) {
            const int s = b % C::STAGES;
            ok = mbar_wait(smem_u32(&bar_full[s]), (b / C::STAGES) & 1, status, &dead, kErrTmaWait);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a = smem0 + s * C::STAGE_BYTES, w = a + C::A_BYTES;
#pragma unroll
            for (int kc = 0; kc < C::NKC; ++kc)
#pragma unroll
                for (int ks = 0; ks < C::KC / 16; ++ks) {
                    const uint64_t ad = make_smem_desc(a + kc * C::A_CHUNK + ks * 32, 16,
                                                       8 * C::SWZ_BYTES, C::LAYOUT);
                    const uint64_t bd = make_smem_desc(w + kc * C::B_CHUNK + ks * 32, 16,
                                                       8 * C::SWZ_BYTES, C::LAYOUT);
                    mma_f16_ss(tmem_base + b * C::NJ, ad, bd, idesc, (kc | ks) != 0);
                }
            mma_commit(smem_u32(&bar_empty[s]));
        }
        mma_commit(smem_u32(&bar_accum));
    }
    __syncwarp();

    // epilogue: thread = token row = TMEM lane
    const bool have = mbar_wait(smem_u32(&bar_accum), 0, status, &dead, kErrMmaWait);
    tc_fence_after();
    const long long t = t0 + threadIdx.x;
    const uint32_t lane_base = tmem_base + ((uint32_t)(warp * 32) << 16);
    if (have && natural) {
        // no permutation: the NJ results of block b are contiguous, out[t][(b0+b)*m + e0 ..]
        for (int b = 0; b < C::NB; ++b) {
#pragma unroll
            for (int ec = 0; ec < C::NJ / 16; ++ec) {
                uint32_t v[16];
                tmem_ld16(lane_base + b * C::NJ + ec * 16, v);
                tmem_ld_wait();
                if (t < tokens) {
                    uint4 o0, o1;
                    o0.x = pack_bf16(__uint_as_float(v[0]), __uint_as_float(v[1]));
                    o0.y = pack_bf16(__uint_as_float(v[2]), __uint_as_float(v[3]));
                    o0.z = pack_bf16(__uint_as_float(v[4]), __uint_as_float(v[5]));
                    o0.w = pack_bf16(__uint_as_float(v[6]), __uint_as_float(v[7]));
                    o1.x = pack_bf16(__uint_as_float(v[8]), __uint_as_float(v[9]));
                    o1.y = pack_bf16(__uint_as_float(v[10]), __uint_as_float(v[11]));
                    o1.z = pack_bf16(__uint_as_float(v[12]), __uint_as_float(v[13]));
                    o1.w = pack_bf16(__uint_as_float(v[14]), __uint_as_float(v[15]));
                    uint4 *dst = reinterpret_cast<uint4 *>(out + (size_t)t * n + (b0 + b) * M + e0 + ec * 16);
                    dst[0] = o0;
                    dst[1] = o1;
                }
            }
        }
    } else if (have) {
        for (int ec = 0; ec < C::NJ / 4; ++ec) {
            uint32_t v[C::NB][4];
#pragma unroll
            for (int b = 0; b < C::NB; ++b) tmem_ld4(lane_base + b * C::NJ + ec * 4, v[b]);
            tmem_ld_wait();
            if (t < tokens) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int col = (e0 + ec * 4 + q) * M + b0;
                    float f[16];
#pragma unroll
                    for (int b = 0; b < 16; ++b) f[b] = __uint_as_float(v[b][q]);
                    if (bias) {
                        const uint4 bv0 = *reinterpret_cast<const uint4 *>(bias + col);
                        const uint4 bv1 = *reinterpret_cast<const uint4 *>(bias + col + 8);
                        const uint32_t bw[8] = {bv0.x, bv0.y, bv0.z, bv0.w, bv1.x, bv1.y, bv1.z, bv1.w};
#pragma unroll
                        for (int b = 0; b < 8; ++b) {
                            f[2 * b] += __uint_as_float(bw[b] << 16);
                            f[2 * b + 1] += __uint_as_float(bw[b] & 0xFFFF0000u);
                        }
                    }
                    if (gelu) {
#pragma unroll
                        for (int b = 0; b < 16; ++b) f[b] = gelu_erf(f[b]);
                    }
                    uint4 o0, o1;
                    o0.x = pack_bf16(f[0], f[1]);
                    o0.y = pack_bf16(f[2], f[3]);
                    o0.z = pack_bf16(f[4], f[5]);
                    o0.w = pack_bf16(f[6], f[7]);
                    o1.x = pack_bf16(f[8], f[9]);
                    o1.y = pack_bf16(f[10], f[11]);
                    o1.z = pack_bf16(f[12], f[13]);
                    o1.w = pack_bf16(f[14], f[15]);
                    uint4 *dst = reinterpret_cast<uint4 *>(out + (size_t)t * n + col);
                    dst[0] = o0;
                    dst[1] = o1;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, C::TMEM_COLS);
}

template <int M>
int launch_tc_stage(const void *in, const void *W, void *out, const void *bias, int gelu, int natural,
                    int64_t tokens, unsigned *status, cudaStream_t s)
{
    using C = StageCfg<M>;
    if (tokens == 0) return MONARCH_OK;
    CUtensorMap tm_in, tm_w;
    MONARCH_TRY(encode_tmap_2d(&tm_in, in, (uint64_t)tokens, (uint64_t)M * M, (uint64_t)M * M * 2,
                               C::TOK, C::KC, C::SWZ_BYTES));
    MONARCH_TRY(encode_tmap_2d(&tm_w, W, (uint64_t)M * M, M, (uint64_t)M * 2, C::NJ, C::KC,
                               C::SWZ_BYTES));
    auto kern = tc_stage_kernel<M>;
    MONARCH_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    dim3 grid((unsigned)((tokens + C::TOK - 1) / C::TOK), M / C::NB, M / C::NJ);
    kern<<<grid, 128, C::SMEM_BYTES, s>>>(tm_in, tm_w, (__nv_bfloat16 *)out,
                                          (const __nv_bfloat16 *)bias, gelu, natural, tokens, status);
    note_launch();
    MONARCH_CUDA_TRY(cudaGetLastError());
    return MONARCH_OK;
}

size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }

}  // namespace

int tc_stage(int m, const void *in, const void *W, void *out, const void *bias, int gelu,
             int64_t tokens, unsigned *status, cudaStream_t s, int natural)
{
    switch (m) {
        case 32:  return launch_tc_stage<32>(in, W, out, bias, gelu, natural, tokens, status, s);
        case 64:  return launch_tc_stage<64>(in, W, out, bias, gelu, natural, tokens, status, s);
        case 128: return launch_tc_stage<128>(in, W, out, bias, gelu, natural, tokens, status, s);
    }
    return MONARCH_ERR_UNSUPPORTED;
}

// ---- host: tensor-map encoder through the driver entry point (no link-time libcuda) ----
typedef CUresult (*tmap_encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

static int tmap_encoder(tmap_encode_fn *out)
{
    static tmap_encode_fn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        MONARCH_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q));
        if (!p || q != cudaDriverEntryPointSuccess) return MONARCH_ERR_CUDA;
        fn = (tmap_encode_fn)p;
    }
    *out = fn;
    return MONARCH_OK;
}

int encode_tmap_2d(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols,
                   uint64_t row_stride_bytes, uint32_t box_rows, uint32_t box_cols,
                   uint32_t swizzle_bytes)
{
    tmap_encode_fn fn;
    MONARCH_TRY(tmap_encoder(&fn));
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_stride_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : swizzle_bytes == 64  ? CU_TENSOR_MAP_SWIZZLE_64B
                                : swizzle_bytes == 32  ? CU_TENSOR_MAP_SWIZZLE_32B
                                                       : CU_TENSOR_MAP_SWIZZLE_NONE;
    const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims,
                          strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MONARCH_OK : MONARCH_ERR_CUDA;
}

int encode_tmap_nd(CUtensorMap *out, const void *base, int elem_bytes, int rank, const uint64_t *dims,
                   const uint64_t *strides_bytes, const uint32_t *box, uint32_t swizzle_bytes)
{
    tmap_encode_fn fn;
    MONARCH_TRY(tmap_encoder(&fn));
    if (rank < 1 || rank > 5) return MONARCH_ERR_INVALID_ARG;
    cuuint64_t d[5], st[4];
    cuuint32_t b[5], es[5];
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) st[i] = strides_bytes[i];
    const CUtensorMapDataType dt = elem_bytes == 8 ? CU_TENSOR_MAP_DATA_TYPE_UINT64
                                 : elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                                   : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const CUresult r = fn(out, dt, (cuuint32_t)rank, const_cast<void *>(base), d, st, b, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE,
                          swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                          : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE,
                          swizzle_bytes == 128 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MONARCH_OK : MONARCH_ERR_CUDA;
}

}  // namespace tc

// Forward pass and feed-forward block as chains of tensor-core stages (bf16, m >= 32); same
// workspace layout as the CUDA-core staged family.
int tc_staged_fwd(const void *x, const void *L, const void *R, void *y, int64_t tokens, int m,
                  void *ws, cudaStream_t s)
{
    if (m == 128) return chain_fwd_m128(x, L, R, y, tokens, ws, s);          // workspace: two plane buffers
    unsigned *status = (unsigned *)ws;
    void *u = (char *)ws + MONARCH_STATUS_BYTES;
    MONARCH_TRY(tc::tc_stage(m, x, R, u, nullptr, 0, tokens, status, s));
    return tc::tc_stage(m, u, L, y, nullptr, 0, tokens, status, s);
}

int tc_staged_mlp_fwd(const void *x, const void *L1, const void *R1, const void *b1, const void *L2,
                      const void *R2, const void *b2, void *y, int64_t tokens, int m, void *ws,
                      cudaStream_t s)
{
    unsigned *status = (unsigned *)ws;
    const size_t act = tc::align256((size_t)tokens * m * m * 2);
    char *base = (char *)ws + MONARCH_STATUS_BYTES;
    void *w = base, *h = base + act;
    MONARCH_TRY(tc::tc_stage(m, x, R1, w, nullptr, 0, tokens, status, s));
    MONARCH_TRY(tc::tc_stage(m, w, L1, h, b1, 1, tokens, status, s));
    MONARCH_TRY(tc::tc_stage(m, h, R2, w, nullptr, 0, tokens, status, s));
    return tc::tc_stage(m, w, L2, y, b2, 0, tokens, status, s);
}

}  // namespace monarch
