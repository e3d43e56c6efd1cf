// C-ABI entry points of libmonarch: argument validation and dispatch.  No arithmetic here.
#include <atomic>
#include <cstdlib>

#include "common.cuh"

namespace monarch {

static std::atomic<uint64_t> g_launches{0};
static std::atomic<int> g_impl{MONARCH_IMPL_AUTO};
static std::atomic<int> g_fixed_order{0};     // monarch_set_deterministic

void note_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int current_device_sms(int *sms)
{
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cache[kMaxDevices];          // zero-initialised: 0 = not yet queried
    int dev = 0;
    MONARCH_CUDA_TRY(cudaGetDevice(&dev));
    int v = dev < kMaxDevices ? cache[dev].load(std::memory_order_relaxed) : 0;
    if (v == 0) {
        MONARCH_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev));
        if (dev < kMaxDevices) cache[dev].store(v, std::memory_order_relaxed);
    }
    *sms = v;
    return MONARCH_OK;
}

namespace {

bool aligned(const void *p, size_t a) { return ((uintptr_t)p & (a - 1)) == 0; }
size_t esize(int dtype) { return dtype == MONARCH_F32 ? 4 : 2; }

struct Range {
    const void *p;
    size_t bytes;
};

bool overlap(const Range &a, const Range &b)
{
    if (!a.p || !b.p || a.bytes == 0 || b.bytes == 0) return false;
    const uintptr_t a0 = (uintptr_t)a.p, a1 = a0 + a.bytes;
    const uintptr_t b0 = (uintptr_t)b.p, b1 = b0 + b.bytes;
    return a0 < b1 && b0 < a1;
}

// Shape / enum checks shared by every call.
int check_shape(int64_t tokens, int32_t n, int32_t m, int dtype)
{
    if (tokens < 0 || n <= 0 || m <= 0) return MONARCH_ERR_INVALID_ARG;
    if (tokens > ((int64_t)1 << 40)) return MONARCH_ERR_INVALID_ARG;        // keeps tokens * n * 4 inside 64 bits
    if ((int64_t)m * m != (int64_t)n) return MONARCH_ERR_INVALID_ARG;
    if (dtype != MONARCH_F32 && dtype != MONARCH_BF16) return MONARCH_ERR_INVALID_ARG;
    if (m != 16 && m != 32 && m != 64 && m != 128) return MONARCH_ERR_UNSUPPORTED;
    return MONARCH_OK;
}

// Sizes of the general (rectangular) multiply.
int check_rect(int64_t tokens, int32_t q, int32_t b1, int32_t b, int32_t r, int dtype)
{
    if (tokens < 0 || q <= 0 || b1 <= 0 || b <= 0 || r <= 0) return MONARCH_ERR_INVALID_ARG;
    if (dtype != MONARCH_F32 && dtype != MONARCH_BF16) return MONARCH_ERR_INVALID_ARG;
    const int64_t lim = 16384, row = (int64_t)1 << 24;
    if (q > lim || b1 > lim || b > lim || r > lim) return MONARCH_ERR_UNSUPPORTED;
    if ((int64_t)q * b1 > row || (int64_t)q * b > row || (int64_t)r * b > row) return MONARCH_ERR_UNSUPPORTED;
    return MONARCH_OK;
}

// Inputs and outputs: non-null, 16-byte aligned; no output overlaps an input, another
// output or the workspace.
int check_buffers(const Range *in, int n_in, const Range *out, int n_out, const void *ws,
                  size_t ws_bytes, size_t ws_need)
{
    for (int i = 0; i < n_in; ++i)
        if (!in[i].p || !aligned(in[i].p, 16)) return MONARCH_ERR_INVALID_ARG;
    for (int i = 0; i < n_out; ++i)
        if (!out[i].p || !aligned(out[i].p, 16)) return MONARCH_ERR_INVALID_ARG;
    if (!ws || !aligned(ws, 256) || ws_need == 0 || ws_bytes < ws_need) return MONARCH_ERR_WORKSPACE;
    const Range w = {ws, ws_bytes};
    for (int o = 0; o < n_out; ++o) {
        for (int i = 0; i < n_in; ++i)
            if (overlap(out[o], in[i])) return MONARCH_ERR_INVALID_ARG;
        for (int p = o + 1; p < n_out; ++p)
            if (overlap(out[o], out[p])) return MONARCH_ERR_INVALID_ARG;
        if (overlap(out[o], w)) return MONARCH_ERR_INVALID_ARG;
    }
    for (int i = 0; i < n_in; ++i)
        if (overlap(in[i], w)) return MONARCH_ERR_INVALID_ARG;
    return MONARCH_OK;
}

enum Family { kSimt = 0, kFused = 1, kTcStaged = 2, kNone = -1 };

// true when the fused tensor-core family has a kernel for (op, m, dtype)
bool fused_available(int op, int m, int dtype)
{
#ifdef MONARCH_TRACE
    static const bool off = getenv("MONARCH_NO_FUSED") != nullptr;   // debug builds: stage chain, for comparison
#else
    constexpr bool off = false;
#endif
    if (off || dtype != MONARCH_BF16) return false;
    return m == 64 || (m == 32 && op == MONARCH_OP_FWD);   // m = 64: every op; m = 32: forward
}

// true when the call can run as a chain of tensor-core stages through the workspace
bool tc_staged_available(int op, int m, int dtype)
{
    if (dtype != MONARCH_BF16 || m < 32) return false;
    if (op == MONARCH_OP_FWD || op == MONARCH_OP_MLP_FWD || op == MONARCH_OP_BWD_DX) return true;
    return m == 32 || m == 64 || m == 128;      // dL, dR: the token-reduction kernel works on 128-column windows
}

// kernel family for a call under the current selection
int pick(int op, int m, int dtype)
{
    const int impl = g_impl.load(std::memory_order_relaxed);
    const bool f = fused_available(op, m, dtype);
    if (impl == MONARCH_IMPL_STAGED) return kSimt;
    if (impl == MONARCH_IMPL_FUSED) return f ? kFused : kNone;
    if (f) return kFused;
    return tc_staged_available(op, m, dtype) ? kTcStaged : kSimt;
}

// Workspace of monarch_mlp_bwd: [backward workspace (status word first)][forward workspace][a][h][dh]
struct MlpBwdLayout {
    size_t ws_b, ws_f, act, off_f, off_a, off_h, off_dh, total;
};

size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }

MlpBwdLayout mlp_bwd_layout(int64_t tokens, int32_t n, int32_t m, int dtype)
{
    MlpBwdLayout l;
    l.ws_b = round256(monarch_workspace_bytes(MONARCH_OP_BWD, tokens, n, m, dtype));
    l.ws_f = round256(monarch_workspace_bytes(MONARCH_OP_FWD, tokens, n, m, dtype));
    l.act = round256((size_t)tokens * n * esize(dtype));
    l.off_f = l.ws_b;
    l.off_a = l.off_f + l.ws_f;
    l.off_h = l.off_a + l.act;
    l.off_dh = l.off_h + l.act;
    l.total = l.off_dh + l.act;
    return l;
}

}  // namespace
}  // namespace monarch

using namespace monarch;

extern "C" {

size_t monarch_workspace_bytes(int op, int64_t tokens, int32_t n, int32_t m, int dtype)
{
    if (op < MONARCH_OP_FWD || op > MONARCH_OP_CPLX) return 0;
    if (check_shape(tokens, n, m, dtype) != MONARCH_OK) return 0;
    if (op == MONARCH_OP_CPLX) {
        // [inner workspace for 2 * tokens rows][four results of 2 * tokens rows]
        const size_t f = monarch_workspace_bytes(MONARCH_OP_FWD, 2 * tokens, n, m, dtype);
        const size_t b = monarch_workspace_bytes(MONARCH_OP_BWD_DX, 2 * tokens, n, m, dtype);
        if (f == 0 || b == 0) return 0;
        return round256(f > b ? f : b) + 4 * round256((size_t)2 * tokens * n * esize(dtype));
    }
    if (op == MONARCH_OP_MLP_BWD) {
        const MlpBwdLayout lay = mlp_bwd_layout(tokens, n, m, dtype);
        return lay.ws_b == 0 || lay.ws_f == 0 ? 0 : lay.total;
    }
    const int which = pick(op, m, dtype);
    if (which < 0) return 0;
    // the fused m = 64 kernels keep one dependency counter per 64-token tile in 64 KB: beyond 2^20 tokens the calls
    // refuse, and so does this query (shard the tokens)
    if (which == kFused && m == 64 && tokens > ((int64_t)1 << 20)) return 0;
    if (which == kTcStaged && op != MONARCH_OP_FWD && op != MONARCH_OP_MLP_FWD)
        return tc_staged_bwd_workspace_bytes(tokens, m, op != MONARCH_OP_BWD_DX && g_fixed_order.load(std::memory_order_relaxed) != 0);
    if (which == kTcStaged && op == MONARCH_OP_FWD && m == 128) return chain_fwd_m128_workspace_bytes(tokens);
    if (op == MONARCH_OP_BWD) {
        if (which == kFused) return fused_bwd_m64_workspace_bytes(tokens, g_fixed_order.load(std::memory_order_relaxed) != 0);
        const size_t a = staged_workspace_bytes(MONARCH_OP_BWD_DX, tokens, n, m, dtype);
        const size_t b = staged_workspace_bytes(MONARCH_OP_BWD_DW, tokens, n, m, dtype);
        return a > b ? a : b;
    }
    if (which == kFused)
        return m == 32                   ? (size_t)MONARCH_STATUS_BYTES
               : op == MONARCH_OP_MLP_FWD ? fused_mlp_fwd_m64_workspace_bytes(tokens)
               : op == MONARCH_OP_FWD    ? fused_fwd_m64_workspace_bytes(tokens)
               : op == MONARCH_OP_BWD_DX ? fused_bwd_dx_m64_workspace_bytes(tokens)
                                         : fused_bwd_dw_m64_workspace_bytes(tokens, g_fixed_order.load(std::memory_order_relaxed) != 0);
    return staged_workspace_bytes(op, tokens, n, m, dtype);
}

int monarch_fwd(const void *x, const void *L, const void *R, void *y, int64_t tokens, int32_t n,
                int32_t m, int dtype, void *workspace, size_t workspace_bytes, void *stream)
{
    MONARCH_TRY(check_shape(tokens, n, m, dtype));
    const size_t act = (size_t)tokens * n * esize(dtype), wb = (size_t)n * m * esize(dtype);
    const Range in[] = {{x, act}, {L, wb}, {R, wb}};
    const Range out[] = {{y, act}};
    const int which = pick(MONARCH_OP_FWD, m, dtype);
    if (which < 0) return MONARCH_ERR_UNSUPPORTED;
    MONARCH_TRY(check_buffers(in, 3, out, 1, workspace, workspace_bytes,
                              monarch_workspace_bytes(MONARCH_OP_FWD, tokens, n, m, dtype)));
    if (which == kFused)
        return m == 32 ? fused_fwd_m32(x, L, R, y, tokens, workspace, (cudaStream_t)stream)
                       : fused_fwd_m64(x, L, R, y, tokens, workspace, (cudaStream_t)stream);
    if (which == kTcStaged) return tc_staged_fwd(x, L, R, y, tokens, m, workspace, (cudaStream_t)stream);
    // the automatic choice runs m = 16 in one launch; MONARCH_IMPL_STAGED keeps the two-launch chain
    if (m == 16 && g_impl.load(std::memory_order_relaxed) == MONARCH_IMPL_AUTO)
        return fused_fwd_m16(x, L, R, y, tokens, dtype, (cudaStream_t)stream);
    return staged_fwd(x, L, R, y, tokens, m, dtype, workspace, (cudaStream_t)stream);
}

int monarch_bwd_dx(const void *dy, const void *L, const void *R, void *dx, int64_t tokens,
                   int32_t n, int32_t m, int dtype, void *workspace, size_t workspace_bytes,
                   void *stream)
{
    MONARCH_TRY(check_shape(tokens, n, m, dtype));
    const size_t act = (size_t)tokens * n * esize(dtype), wb = (size_t)n * m * esize(dtype);
    const Range in[] = {{dy, act}, {L, wb}, {R, wb}};
    const Range out[] = {{dx, act}};
    const int which = pick(MONARCH_OP_BWD_DX, m, dtype);
    if (which < 0) return MONARCH_ERR_UNSUPPORTED;
    MONARCH_TRY(check_buffers(in, 3, out, 1, workspace, workspace_bytes,
                              monarch_workspace_bytes(MONARCH_OP_BWD_DX, tokens, n, m, dtype)));
    if (which == kFused)
        return fused_bwd_dx_m64(dy, L, R, dx, tokens, workspace, (cudaStream_t)stream);
    if (which == kTcStaged)
        return tc_staged_bwd(nullptr, dy, L, R, dx, nullptr, nullptr, 0, 1, 0, tokens, m, workspace,
                             (cudaStream_t)stream);
    return staged_bwd_dx(dy, L, R, dx, tokens, m, dtype, workspace, (cudaStream_t)stream);
}

int monarch_bwd_dw(const void *x, const void *dy, const void *L, const void *R, float *dL,
                   float *dR, int accumulate, int64_t tokens, int32_t n, int32_t m, int dtype,
                   void *workspace, size_t workspace_bytes, void *stream)
{
    MONARCH_TRY(check_shape(tokens, n, m, dtype));
    if (accumulate != 0 && accumulate != 1) return MONARCH_ERR_INVALID_ARG;
    const size_t act = (size_t)tokens * n * esize(dtype), wb = (size_t)n * m * esize(dtype);
    const size_t gb = (size_t)n * m * sizeof(float);
    const Range in[] = {{x, act}, {dy, act}, {L, wb}, {R, wb}};
    const Range out[] = {{dL, gb}, {dR, gb}};
    const int which = pick(MONARCH_OP_BWD_DW, m, dtype);
    if (which < 0) return MONARCH_ERR_UNSUPPORTED;
    MONARCH_TRY(check_buffers(in, 4, out, 2, workspace, workspace_bytes,
                              monarch_workspace_bytes(MONARCH_OP_BWD_DW, tokens, n, m, dtype)));
    if (which == kFused)
        return fused_bwd_dw_m64(x, dy, L, R, dL, dR, accumulate, tokens, workspace, (cudaStream_t)stream,
                                g_fixed_order.load(std::memory_order_relaxed) != 0);
    if (which == kTcStaged)
        return tc_staged_bwd(x, dy, L, R, nullptr, dL, dR, accumulate, 0, 1, tokens, m, workspace,
                             (cudaStream_t)stream, nullptr, g_fixed_order.load(std::memory_order_relaxed) != 0);
    return staged_bwd_dw(x, dy, L, R, dL, dR, accumulate, tokens, m, dtype, workspace,
                         (cudaStream_t)stream);
}

int monarch_bwd(const void *x, const void *dy, const void *L, const void *R, const void *fwd_workspace,
                void *dx, float *dL, float *dR, int accumulate, int64_t tokens, int32_t n, int32_t m,
                int dtype, void *workspace, size_t workspace_bytes, void *stream)
{
    MONARCH_TRY(check_shape(tokens, n, m, dtype));
    if (accumulate != 0 && accumulate != 1) return MONARCH_ERR_INVALID_ARG;
    if (fwd_workspace != nullptr && fwd_workspace == workspace) return MONARCH_ERR_INVALID_ARG;
    const size_t act = (size_t)tokens * n * esize(dtype), wb = (size_t)n * m * esize(dtype);
    const size_t gb = (size_t)n * m * sizeof(float);
    const Range in[] = {{x, act}, {dy, act}, {L, wb}, {R, wb}};
    const Range out[] = {{dx, act}, {dL, gb}, {dR, gb}};
    const int which = pick(MONARCH_OP_BWD, m, dtype);
    if (which < 0) return MONARCH_ERR_UNSUPPORTED;
    MONARCH_TRY(check_buffers(in, 4, out, 3, workspace, workspace_bytes,
                              monarch_workspace_bytes(MONARCH_OP_BWD, tokens, n, m, dtype)));
    cudaStream_t s = (cudaStream_t)stream;
    if (which == kFused) {
        const bool saved = fwd_workspace != nullptr && pick(MONARCH_OP_FWD, m, dtype) == kFused;
        return fused_bwd_m64(x, dy, L, R, saved ? fused_fwd_m64_saved_u(fwd_workspace) : nullptr, dx, dL,
                             dR, accumulate, tokens, workspace, s, g_fixed_order.load(std::memory_order_relaxed) != 0);
    }
    if (which == kTcStaged) {
        const bool saved = fwd_workspace != nullptr && m == 128 && pick(MONARCH_OP_FWD, m, dtype) == kTcStaged;
        return tc_staged_bwd(x, dy, L, R, dx, dL, dR, accumulate, 1, 1, tokens, m, workspace, s,
                             saved ? chain_fwd_m128_saved_u(fwd_workspace, tokens) : nullptr,
                             g_fixed_order.load(std::memory_order_relaxed) != 0);
    }
    MONARCH_TRY(staged_bwd_dx(dy, L, R, dx, tokens, m, dtype, workspace, s));
    return staged_bwd_dw(x, dy, L, R, dL, dR, accumulate, tokens, m, dtype, workspace, s);
}

int monarch_mlp_fwd(const void *x, const void *L1, const void *R1, const void *b1, const void *L2,
                    const void *R2, const void *b2, void *y, int64_t tokens, int32_t n, int32_t m,
                    int dtype, void *workspace, size_t workspace_bytes, void *stream)
{
    MONARCH_TRY(check_shape(tokens, n, m, dtype));
    const size_t act = (size_t)tokens * n * esize(dtype), wb = (size_t)n * m * esize(dtype);
    const size_t bb = (size_t)n * esize(dtype);
    const Range in[] = {{x, act}, {L1, wb}, {R1, wb}, {b1, bb}, {L2, wb}, {R2, wb}, {b2, bb}};
    const Range out[] = {{y, act}};
    const int which = pick(MONARCH_OP_MLP_FWD, m, dtype);
    if (which < 0) return MONARCH_ERR_UNSUPPORTED;
    MONARCH_TRY(check_buffers(in, 7, out, 1, workspace, workspace_bytes,
                              monarch_workspace_bytes(MONARCH_OP_MLP_FWD, tokens, n, m, dtype)));
    if (which == kFused)
        return fused_mlp_fwd_m64(x, L1, R1, b1, L2, R2, b2, y, tokens, workspace, (cudaStream_t)stream);
    if (which == kTcStaged)
        return tc_staged_mlp_fwd(x, L1, R1, b1, L2, R2, b2, y, tokens, m, workspace,
                                 (cudaStream_t)stream);
    return staged_mlp_fwd(x, L1, R1, b1, L2, R2, b2, y, tokens, m, dtype, workspace,
                          (cudaStream_t)stream);
}

int monarch_mlp_bwd(const void *x, const void *dy, const void *L1, const void *R1, const void *b1,
                    const void *L2, const void *R2, void *dx, float *dL1, float *dR1, float *db1,
                    float *dL2, float *dR2, float *db2, int accumulate, int64_t tokens, int32_t n,
                    int32_t m, int dtype, void *workspace, size_t workspace_bytes, void *stream)
{
    MONARCH_TRY(check_shape(tokens, n, m, dtype));
    if (accumulate != 0 && accumulate != 1) return MONARCH_ERR_INVALID_ARG;
    const size_t act = (size_t)tokens * n * esize(dtype), wb = (size_t)n * m * esize(dtype);
    const size_t bb = (size_t)n * esize(dtype), gb = (size_t)n * m * sizeof(float);
    const size_t gbias = (size_t)n * sizeof(float);
    const Range in[] = {{x, act}, {dy, act}, {L1, wb}, {R1, wb}, {b1, bb}, {L2, wb}, {R2, wb}};
    const Range out[] = {{dx, act}, {dL1, gb}, {dR1, gb}, {db1, gbias}, {dL2, gb}, {dR2, gb}, {db2, gbias}};
    const MlpBwdLayout lay = mlp_bwd_layout(tokens, n, m, dtype);
    if (lay.ws_b == 0 || lay.ws_f == 0) return MONARCH_ERR_UNSUPPORTED;
    MONARCH_TRY(check_buffers(in, 7, out, 7, workspace, workspace_bytes, lay.total));
    cudaStream_t s = (cudaStream_t)stream;
    if (!accumulate) {
        MONARCH_CUDA_TRY(cudaMemsetAsync(db1, 0, gbias, s));
        MONARCH_CUDA_TRY(cudaMemsetAsync(db2, 0, gbias, s));
    }
    char *ws = (char *)workspace;
    void *ws_b = ws, *ws_f = ws + lay.off_f;
    void *a = ws + lay.off_a, *h = ws + lay.off_h, *dh = ws + lay.off_dh;
    // the inner forward workspace starts with its own status word and tile counters
    MONARCH_TRY(monarch_workspace_init(ws_f, lay.ws_f, stream));
    // a = M1 x + b1: the fused m = 64 forward adds the bias in its epilogue, the others leave it to the
    // elementwise kernels (a then holds M1 x)
    const bool bias_in_a = pick(MONARCH_OP_FWD, m, dtype) == kFused && m == 64;
    if (bias_in_a)
        MONARCH_TRY(fused_fwd_bias_m64(x, L1, R1, b1, 0, a, tokens, ws_f, s));
    else
        MONARCH_TRY(monarch_fwd(x, L1, R1, a, tokens, n, m, dtype, ws_f, lay.ws_f, stream));
    const void *b1_late = bias_in_a ? nullptr : b1;
    MONARCH_TRY(mlp_act(a, b1_late, h, tokens, n, dtype, s));
    // second matrix: dh = M2^T dy and its block gradients, input h
    MONARCH_TRY(monarch_bwd(h, dy, L2, R2, nullptr, dh, dL2, dR2, accumulate, tokens, n, m, dtype, ws_b,
                            lay.ws_b, stream));
    MONARCH_TRY(mlp_dact(dh, a, b1_late, dy, db1, db2, tokens, n, dtype, s));
    // first matrix: dx = M1^T da and its block gradients; u = P^T R1 x is still in the forward workspace
    MONARCH_TRY(monarch_bwd(x, dh, L1, R1, ws_f, dx, dL1, dR1, accumulate, tokens, n, m, dtype, ws_b, lay.ws_b,
                            stream));
    return merge_status((unsigned *)ws_b, (unsigned *)ws_f, s);
}

size_t monarch_rect_workspace_bytes(int64_t tokens, int32_t q, int32_t b1, int32_t b, int32_t r, int dtype)
{
    if (check_rect(tokens, q, b1, b, r, dtype) != MONARCH_OK) return 0;
    return rect_workspace_bytes(tokens, q, b, dtype);
}

int monarch_rect_fwd(const void *x, const void *L, const void *R, void *y, int64_t tokens, int32_t q,
                     int32_t b1, int32_t b, int32_t r, int dtype, void *workspace,
                     size_t workspace_bytes, void *stream)
{
    MONARCH_TRY(check_rect(tokens, q, b1, b, r, dtype));
    const size_t es = esize(dtype);
    const Range in[] = {{x, (size_t)tokens * q * b1 * es}, {L, (size_t)b * r * q * es}, {R, (size_t)q * b * b1 * es}};
    const Range out[] = {{y, (size_t)tokens * r * b * es}};
    MONARCH_TRY(check_buffers(in, 3, out, 1, workspace, workspace_bytes, rect_workspace_bytes(tokens, q, b, dtype)));
    cudaStream_t s = (cudaStream_t)stream;
    void *u = (char *)workspace + MONARCH_STATUS_BYTES;
    unsigned *status = (unsigned *)workspace;
    const bool fast = g_impl.load(std::memory_order_relaxed) != MONARCH_IMPL_STAGED;
    // large bf16 blocks: stage 1 (nearly all the FLOPs when q is small) on the tensor cores
    if (fast && rect_stage1_tc_available(q, b1, b, dtype))
        MONARCH_TRY(rect_stage1_tc(x, R, u, tokens, q, b1, b, status, s));
    else
        MONARCH_TRY(rect_stage1_simt(x, R, u, tokens, q, b1, b, dtype, 0, s));
    if (fast && rect_stage2_stream_available(q, b, r, dtype))
        return rect_stage2_stream(u, L, y, tokens, q, b, r, 0, status, s);
    return rect_stage2_simt(u, L, y, tokens, q, b, r, dtype, 0, s);
}

size_t monarch_rectw_workspace_bytes(int64_t tokens, int32_t q, int32_t b1, int32_t b2, int32_t b3, int32_t r, int dtype)
{
    if (check_rect(tokens, q, b1, b2, 1, dtype) != MONARCH_OK || check_rect(tokens, q, 1, b3, r, dtype) != MONARCH_OK) return 0;
    return rectw_workspace_bytes(tokens, q, b2, b3, r, dtype);
}

size_t monarch_rectw_bwd_workspace_bytes(int64_t tokens, int32_t q, int32_t b1, int32_t b2, int32_t b3, int32_t r, int dtype)
{
    if (check_rect(tokens, q, b1, b2, 1, dtype) != MONARCH_OK || check_rect(tokens, q, 1, b3, r, dtype) != MONARCH_OK) return 0;
    return rectw_bwd_workspace_bytes(tokens, q, b2, b3, r, dtype);
}

int monarch_rectw_fwd(const void *x, const void *L, const void *R, void *y, int64_t tokens, int32_t q, int32_t b1,
                      int32_t b2, int32_t b3, int32_t r, int dtype, void *workspace, size_t workspace_bytes, void *stream)
{
    MONARCH_TRY(check_rect(tokens, q, b1, b2, 1, dtype));
    MONARCH_TRY(check_rect(tokens, q, 1, b3, r, dtype));
    const size_t es = esize(dtype), bmax = b2 > b3 ? b2 : b3;
    const Range in[] = {{x, (size_t)tokens * q * b1 * es}, {L, (size_t)r * q * bmax * es}, {R, (size_t)q * b2 * b1 * es}};
    const Range out[] = {{y, (size_t)tokens * r * b3 * es}};
    MONARCH_TRY(check_buffers(in, 3, out, 1, workspace, workspace_bytes, rectw_workspace_bytes(tokens, q, b2, b3, r, dtype)));
    const bool fast = g_impl.load(std::memory_order_relaxed) != MONARCH_IMPL_STAGED;
    return rectw_fwd(x, L, R, y, tokens, q, b1, b2, b3, r, dtype, fast, workspace, (cudaStream_t)stream);
}

int monarch_rectw_bwd(const void *x, const void *dy, const void *L, const void *R, void *dx, float *dL, float *dR,
                      int accumulate, int64_t tokens, int32_t q, int32_t b1, int32_t b2, int32_t b3, int32_t r, int dtype,
                      void *workspace, size_t workspace_bytes, void *stream)
{
    MONARCH_TRY(check_rect(tokens, q, b1, b2, 1, dtype));
    MONARCH_TRY(check_rect(tokens, q, 1, b3, r, dtype));
    if (accumulate != 0 && accumulate != 1) return MONARCH_ERR_INVALID_ARG;
    const size_t es = esize(dtype), bmax = b2 > b3 ? b2 : b3;
    const size_t lb = (size_t)r * q * bmax, rb = (size_t)q * b2 * b1;
    const Range in[] = {{x, (size_t)tokens * q * b1 * es}, {dy, (size_t)tokens * r * b3 * es}, {L, lb * es}, {R, rb * es}};
    const Range out[] = {{dx, (size_t)tokens * q * b1 * es}, {dL, lb * sizeof(float)}, {dR, rb * sizeof(float)}};
    MONARCH_TRY(check_buffers(in, 4, out, 3, workspace, workspace_bytes,
                              rectw_bwd_workspace_bytes(tokens, q, b2, b3, r, dtype)));
    const bool fast = g_impl.load(std::memory_order_relaxed) != MONARCH_IMPL_STAGED;
    return rectw_bwd(x, dy, L, R, dx, dL, dR, accumulate, tokens, q, b1, b2, b3, r, dtype, fast, workspace, (cudaStream_t)stream);
}

size_t monarch_rect_bwd_workspace_bytes(int64_t tokens, int32_t q, int32_t b1, int32_t b, int32_t r, int dtype)
{
    if (check_rect(tokens, q, b1, b, r, dtype) != MONARCH_OK) return 0;
    return MONARCH_STATUS_BYTES + 2 * round256((size_t)tokens * q * b * esize(dtype));      // [status][u][du]
}

int monarch_rect_bwd(const void *x, const void *dy, const void *L, const void *R, const void *fwd_workspace,
                     void *dx, float *dL, float *dR, int accumulate, int64_t tokens, int32_t q, int32_t b1, int32_t b, int32_t r, int dtype,
                     void *workspace, size_t workspace_bytes, void *stream)
{
    MONARCH_TRY(check_rect(tokens, q, b1, b, r, dtype));
    if (accumulate != 0 && accumulate != 1) return MONARCH_ERR_INVALID_ARG;
    if (fwd_workspace != nullptr && (fwd_workspace == workspace || !aligned(fwd_workspace, 256)))
        return MONARCH_ERR_INVALID_ARG;
    const size_t es = esize(dtype);
    const size_t lb = (size_t)b * r * q, rb = (size_t)q * b * b1;
    const Range in[] = {{x, (size_t)tokens * q * b1 * es}, {dy, (size_t)tokens * r * b * es}, {L, lb * es}, {R, rb * es}};
    const Range out[] = {{dx, (size_t)tokens * q * b1 * es}, {dL, lb * sizeof(float)}, {dR, rb * sizeof(float)}};
    MONARCH_TRY(check_buffers(in, 4, out, 3, workspace, workspace_bytes,
                              monarch_rect_bwd_workspace_bytes(tokens, q, b1, b, r, dtype)));
    cudaStream_t s = (cudaStream_t)stream;
    if (!accumulate) {
        MONARCH_CUDA_TRY(cudaMemsetAsync(dL, 0, lb * sizeof(float), s));
        MONARCH_CUDA_TRY(cudaMemsetAsync(dR, 0, rb * sizeof(float), s));
    }
    if (tokens == 0) return MONARCH_OK;
    unsigned *status = (unsigned *)workspace;
    char *u_own = (char *)workspace + MONARCH_STATUS_BYTES;
    char *du = u_own + round256((size_t)tokens * q * b * es);
    const bool fast = g_impl.load(std::memory_order_relaxed) != MONARCH_IMPL_STAGED;
    // u = blockdiag(R) x: what the forward call left in its workspace ([status][u]), else recomputed
    const char *u = fwd_workspace ? (const char *)fwd_workspace + MONARCH_STATUS_BYTES : u_own;
    if (!fwd_workspace) {
        if (fast && rect_stage1_tc_available(q, b1, b, dtype))
            MONARCH_TRY(rect_stage1_tc(x, R, u_own, tokens, q, b1, b, status, s));
        else
            MONARCH_TRY(rect_stage1_simt(x, R, u_own, tokens, q, b1, b, dtype, 0, s));
    }
    // du = L^T dy: stage 2 with the roles of q and r exchanged and the blocks read transposed
    if (fast && rect_stage2_stream_available(r, b, q, dtype))
        MONARCH_TRY(rect_stage2_stream(dy, L, du, tokens, r, b, q, 1, status, s));
    else
        MONARCH_TRY(rect_stage2_simt(dy, L, du, tokens, r, b, q, dtype, 1, s));
    // dx = blockdiag(R)^T du: stage 1 with the roles of b1 and b exchanged and the blocks read transposed
    if (fast && rect_stage1_tc_available(q, b1, b, dtype))
        MONARCH_TRY(rect_stage1_adjoint_tc(du, R, dx, tokens, q, b1, b, status, s));
    else
        MONARCH_TRY(rect_stage1_simt(du, R, dx, tokens, q, b, b1, dtype, 1, s));
    const bool tc_dR = fast && rect_wgrad_R_tc_available(q, b1, b, dtype);
    if (tc_dR) MONARCH_TRY(rect_wgrad_R_tc(du, x, dR, tokens, q, b1, b, status, s));
    const bool stream_dL = fast && rect_stage2_stream_available(q, b, r, dtype);
    if (stream_dL) MONARCH_TRY(rect_dl_stream(dy, u, dL, tokens, q, b, r, status, s));
    return rect_wgrad_simt(x, dy, u, du, dL, dR, tokens, q, b1, b, r, dtype, !stream_dL, !tc_dR, s);
}

int monarch_cplx_fwd(const void *x, const void *L, const void *R, void *y, int adjoint, int64_t tokens,
                     int32_t n, int32_t m, int dtype, void *workspace, size_t workspace_bytes, void *stream)
{
    MONARCH_TRY(check_shape(tokens, n, m, dtype));
    if (adjoint != 0 && adjoint != 1) return MONARCH_ERR_INVALID_ARG;
    const size_t es = esize(dtype), plane = (size_t)tokens * n * es, wplane = (size_t)n * m * es;
    const Range in[] = {{x, 2 * plane}, {L, 2 * wplane}, {R, 2 * wplane}};
    const Range out[] = {{y, 2 * plane}};
    const size_t need = monarch_workspace_bytes(MONARCH_OP_CPLX, tokens, n, m, dtype);
    MONARCH_TRY(check_buffers(in, 3, out, 1, workspace, workspace_bytes, need));
    const size_t res = round256(2 * plane);
    const size_t inner = need - 4 * res;
    char *ws = (char *)workspace;
    void *part[4] = {ws + inner, ws + inner + res, ws + inner + 2 * res, ws + inner + 3 * res};
    const char *Lr = (const char *)L, *Li = Lr + wplane, *Rr = (const char *)R, *Ri = Rr + wplane;
    const char *lsel[4] = {Lr, Li, Lr, Li}, *rsel[4] = {Rr, Ri, Ri, Rr};   // A, B, C, D
    for (int c = 0; c < 4; ++c) {
        // both planes at once: [xr; xi] is 2 * tokens rows
        if (adjoint)
            MONARCH_TRY(monarch_bwd_dx(x, lsel[c], rsel[c], part[c], 2 * tokens, n, m, dtype, ws, inner, stream));
        else
            MONARCH_TRY(monarch_fwd(x, lsel[c], rsel[c], part[c], 2 * tokens, n, m, dtype, ws, inner, stream));
    }
    return cplx_combine(part[0], part[1], part[2], part[3], y, (int64_t)tokens * n, adjoint, dtype,
                        (cudaStream_t)stream);
}

int monarch_dense(const void *L, const void *R, void *M, int32_t n, int32_t m, int dtype, void *stream)
{
    MONARCH_TRY(check_shape(0, n, m, dtype));
    const size_t wb = (size_t)n * m * esize(dtype), mb = (size_t)n * n * esize(dtype);
    const Range in[] = {{L, wb}, {R, wb}};
    const Range out = {M, mb};
    for (const Range &r : in)
        if (!r.p || !aligned(r.p, 16) || overlap(out, r)) return MONARCH_ERR_INVALID_ARG;
    if (!M || !aligned(M, 16)) return MONARCH_ERR_INVALID_ARG;
    return dense_from_factors(L, R, M, m, dtype, (cudaStream_t)stream);
}

int monarch_project(const void *A, void *L, void *R, int32_t n, int32_t m, int dtype,
                    unsigned long long *rotation_count, void *stream)
{
    MONARCH_TRY(check_shape(0, n, m, dtype));
    const size_t wb = (size_t)n * m * esize(dtype), mb = (size_t)n * n * esize(dtype);
    const Range in = {A, mb};
    const Range out[] = {{L, wb}, {R, wb}};
    if (!A || !aligned(A, 16)) return MONARCH_ERR_INVALID_ARG;
    for (const Range &r : out)
        if (!r.p || !aligned(r.p, 16) || overlap(r, in)) return MONARCH_ERR_INVALID_ARG;
    if (overlap(out[0], out[1])) return MONARCH_ERR_INVALID_ARG;
    return project_to_factors(A, L, R, m, dtype, rotation_count, (cudaStream_t)stream);
}

int monarch_workspace_init(void *workspace, size_t workspace_bytes, void *stream)
{
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < MONARCH_STATUS_BYTES)
        return MONARCH_ERR_WORKSPACE;
    // status word plus the dependency counters that follow it (64 KB) where the workspace has them
    const size_t clear = workspace_bytes < MONARCH_STATUS_BYTES + 65536 ? workspace_bytes
                                                                         : MONARCH_STATUS_BYTES + 65536;
    MONARCH_CUDA_TRY(cudaMemsetAsync(workspace, 0, clear, (cudaStream_t)stream));
    return MONARCH_OK;
}

int monarch_last_device_status(void *workspace, void *stream)
{
    if (!workspace || ((uintptr_t)workspace & 255)) return MONARCH_ERR_WORKSPACE;
    unsigned int word = 0;
    cudaStream_t s = (cudaStream_t)stream;
    MONARCH_CUDA_TRY(cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, s));
    MONARCH_CUDA_TRY(cudaStreamSynchronize(s));
    if (word != 0) {
        MONARCH_CUDA_TRY(cudaMemsetAsync(workspace, 0, MONARCH_STATUS_BYTES, s));
        MONARCH_CUDA_TRY(cudaStreamSynchronize(s));
        return MONARCH_ERR_TIMEOUT;
    }
    return MONARCH_OK;
}

int monarch_debug_set_wait_limit(void *workspace, unsigned int microseconds, void *stream)
{
    if (!workspace || ((uintptr_t)workspace & 255)) return MONARCH_ERR_WORKSPACE;
    // pageable source: the copy is staged before the call returns
    MONARCH_CUDA_TRY(cudaMemcpyAsync((char *)workspace + sizeof(unsigned int), &microseconds, sizeof(microseconds),
                                     cudaMemcpyHostToDevice, (cudaStream_t)stream));
    return MONARCH_OK;
}

int monarch_debug_skip_load(int64_t item)
{
    debug_skip_next_plane_load(item);
    return MONARCH_OK;
}

int monarch_set_deterministic(int on)
{
    return g_fixed_order.exchange(on != 0 ? 1 : 0);
}

int monarch_set_impl(int impl)
{
    if (impl < MONARCH_IMPL_AUTO || impl > MONARCH_IMPL_FUSED) return -1;
    return g_impl.exchange(impl);
}

const char *monarch_impl_name(int op, int32_t m, int dtype)
{
    if (op < MONARCH_OP_FWD || op > MONARCH_OP_CPLX) return "unsupported";
    if (check_shape(0, m * m, m, dtype) != MONARCH_OK) return "unsupported";
    if (op == MONARCH_OP_MLP_BWD) op = MONARCH_OP_BWD;      // its Monarch passes are monarch_bwd's
    if (op == MONARCH_OP_CPLX) op = MONARCH_OP_FWD;         // four real forward (or dx) passes
    const int which = pick(op, m, dtype);
    if (which == kSimt && op == MONARCH_OP_FWD && m == 16 &&
        g_impl.load(std::memory_order_relaxed) == MONARCH_IMPL_AUTO)
        return "fused-simt";
    return which < 0 ? "unsupported" : which == kFused ? "fused-tcgen05"
         : which == kTcStaged ? "staged-tcgen05" : "staged-simt";
}

uint64_t monarch_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char *monarch_status_string(int status)
{
    switch (status) {
        case MONARCH_OK: return "ok";
        case MONARCH_ERR_INVALID_ARG: return "invalid argument";
        case MONARCH_ERR_UNSUPPORTED: return "unsupported size or dtype";
        case MONARCH_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case MONARCH_ERR_CUDA: return "CUDA error";
        case MONARCH_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

}  // extern "C"
