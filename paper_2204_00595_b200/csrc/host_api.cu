// Host-buffer entry points: the caller's tensors live in host memory; the library streams them
// through the GPU in token chunks so that the upload of chunk c+1, the kernels of chunk c and the
// download of chunk c-1 overlap on three streams.  All arithmetic is done by the device entry points
// (monarch_fwd / monarch_bwd); nothing is computed on the host.
#include <cstdlib>
#include <new>

#include "common.cuh"

namespace {
constexpr int kBuf = 3;      // chunk buffers in flight

size_t esz(int dtype) { return dtype == MONARCH_F32 ? 4 : 2; }
}  // namespace

struct monarch_host_ctx {
    int64_t max_tokens = 0, chunk = 0;
    int32_t n = 0, m = 0;
    int dtype = 0;
    cudaStream_t s_in = nullptr, s_run = nullptr, s_out = nullptr;
    cudaEvent_t in_ready[kBuf] = {}, out_ready[kBuf] = {}, out_done[kBuf] = {}, w_ready = nullptr;
    char *x[kBuf] = {}, *dy[kBuf] = {}, *y[kBuf] = {}, *dx[kBuf] = {};
    char *L = nullptr, *R = nullptr;
    float *dL = nullptr, *dR = nullptr;
    void *ws = nullptr, *ws_b = nullptr;      // forward workspace (keeps u for the backward call), backward
    size_t ws_bytes = 0, ws_b_bytes = 0;
};

namespace {

void destroy(monarch_host_ctx *c)
{
    if (!c) return;
    for (int i = 0; i < kBuf; ++i) {
        cudaFree(c->x[i]); cudaFree(c->dy[i]); cudaFree(c->y[i]); cudaFree(c->dx[i]);
        if (c->in_ready[i]) cudaEventDestroy(c->in_ready[i]);
        if (c->out_ready[i]) cudaEventDestroy(c->out_ready[i]);
        if (c->out_done[i]) cudaEventDestroy(c->out_done[i]);
    }
    if (c->w_ready) cudaEventDestroy(c->w_ready);
    cudaFree(c->L); cudaFree(c->R); cudaFree(c->dL); cudaFree(c->dR); cudaFree(c->ws); cudaFree(c->ws_b);
    if (c->s_in) cudaStreamDestroy(c->s_in);
    if (c->s_run) cudaStreamDestroy(c->s_run);
    if (c->s_out) cudaStreamDestroy(c->s_out);
    delete c;
}

int run(monarch_host_ctx *c, const void *x, const void *dy, const void *L, const void *R, void *y,
        void *dx, float *dL, float *dR, int64_t tokens, bool backward)
{
    if (!c || !L || !R || tokens < 0 || tokens > c->max_tokens) return MONARCH_ERR_INVALID_ARG;
    if (tokens > 0 && (!x || !y || (backward && (!dy || !dx)))) return MONARCH_ERR_INVALID_ARG;
    if (backward && (!dL || !dR)) return MONARCH_ERR_INVALID_ARG;
    const size_t e = esz(c->dtype), row = (size_t)c->n * e, wb = (size_t)c->n * c->m * e;
    const size_t gb = (size_t)c->n * c->m * sizeof(float);
    MONARCH_CUDA_TRY(cudaMemcpyAsync(c->L, L, wb, cudaMemcpyHostToDevice, c->s_in));
    MONARCH_CUDA_TRY(cudaMemcpyAsync(c->R, R, wb, cudaMemcpyHostToDevice, c->s_in));
    MONARCH_CUDA_TRY(cudaEventRecord(c->w_ready, c->s_in));
    MONARCH_CUDA_TRY(cudaStreamWaitEvent(c->s_run, c->w_ready, 0));
    const int64_t chunks = (tokens + c->chunk - 1) / c->chunk;
    if (backward && chunks == 0) {
        MONARCH_CUDA_TRY(cudaMemsetAsync(c->dL, 0, gb, c->s_run));
        MONARCH_CUDA_TRY(cudaMemsetAsync(c->dR, 0, gb, c->s_run));
    }
    for (int64_t ci = 0; ci < chunks; ++ci) {
        const int b = (int)(ci % kBuf);
        const int64_t t0 = ci * c->chunk, tn = tokens - t0 < c->chunk ? tokens - t0 : c->chunk;
        const size_t off = (size_t)t0 * row, bytes = (size_t)tn * row;
        // the buffers of slot b are free once the download of the chunk that used them is done
        if (ci >= kBuf) MONARCH_CUDA_TRY(cudaStreamWaitEvent(c->s_in, c->out_done[b], 0));
        MONARCH_CUDA_TRY(cudaMemcpyAsync(c->x[b], (const char *)x + off, bytes, cudaMemcpyHostToDevice, c->s_in));
        if (backward)
            MONARCH_CUDA_TRY(cudaMemcpyAsync(c->dy[b], (const char *)dy + off, bytes, cudaMemcpyHostToDevice, c->s_in));
        MONARCH_CUDA_TRY(cudaEventRecord(c->in_ready[b], c->s_in));

        MONARCH_CUDA_TRY(cudaStreamWaitEvent(c->s_run, c->in_ready[b], 0));
        if (ci >= kBuf) MONARCH_CUDA_TRY(cudaStreamWaitEvent(c->s_run, c->out_done[b], 0));
        MONARCH_TRY(monarch_fwd(c->x[b], c->L, c->R, c->y[b], tn, c->n, c->m, c->dtype, c->ws, c->ws_bytes, c->s_run));
        if (backward)
            MONARCH_TRY(monarch_bwd(c->x[b], c->dy[b], c->L, c->R, c->ws, c->dx[b], c->dL, c->dR, ci > 0, tn,
                                    c->n, c->m, c->dtype, c->ws_b, c->ws_b_bytes, c->s_run));
        MONARCH_CUDA_TRY(cudaEventRecord(c->out_ready[b], c->s_run));

        MONARCH_CUDA_TRY(cudaStreamWaitEvent(c->s_out, c->out_ready[b], 0));
        MONARCH_CUDA_TRY(cudaMemcpyAsync((char *)y + off, c->y[b], bytes, cudaMemcpyDeviceToHost, c->s_out));
        if (backward)
            MONARCH_CUDA_TRY(cudaMemcpyAsync((char *)dx + off, c->dx[b], bytes, cudaMemcpyDeviceToHost, c->s_out));
        MONARCH_CUDA_TRY(cudaEventRecord(c->out_done[b], c->s_out));
    }
    if (backward) {
        MONARCH_CUDA_TRY(cudaMemcpyAsync(dL, c->dL, gb, cudaMemcpyDeviceToHost, c->s_run));
        MONARCH_CUDA_TRY(cudaMemcpyAsync(dR, c->dR, gb, cudaMemcpyDeviceToHost, c->s_run));
    }
    MONARCH_CUDA_TRY(cudaStreamSynchronize(c->s_in));
    MONARCH_CUDA_TRY(cudaStreamSynchronize(c->s_out));
    MONARCH_TRY(monarch_last_device_status(c->ws, c->s_run));
    return monarch_last_device_status(c->ws_b, c->s_run);
}

}  // namespace

extern "C" {

int monarch_host_create(monarch_host_ctx **out, int64_t max_tokens, int32_t n, int32_t m, int dtype,
                        int64_t chunk_tokens)
{
    if (!out || max_tokens < 0 || chunk_tokens < 0) return MONARCH_ERR_INVALID_ARG;
    *out = nullptr;
    if (chunk_tokens == 0) {
        // default: about eight chunks, so that uploads and downloads overlap for most of the call (the first upload
        // and the last download cannot), but no smaller than 256 tokens (the kernels' fill and drain) nor larger than 2048
        chunk_tokens = (max_tokens / 8 + 63) / 64 * 64;
        if (chunk_tokens < 256) chunk_tokens = 256;
        if (chunk_tokens > 2048) chunk_tokens = 2048;
    }
    if (chunk_tokens % 64) return MONARCH_ERR_INVALID_ARG;
    if (chunk_tokens > max_tokens && max_tokens > 0) chunk_tokens = (max_tokens + 63) / 64 * 64;
    const size_t wsb = monarch_workspace_bytes(MONARCH_OP_FWD, chunk_tokens, n, m, dtype);
    const size_t wsb_b = monarch_workspace_bytes(MONARCH_OP_BWD, chunk_tokens, n, m, dtype);
    if (wsb == 0 || wsb_b == 0) return MONARCH_ERR_UNSUPPORTED;
    monarch_host_ctx *c = new (std::nothrow) monarch_host_ctx;
    if (!c) return MONARCH_ERR_CUDA;
    c->max_tokens = max_tokens; c->chunk = chunk_tokens; c->n = n; c->m = m; c->dtype = dtype;
    c->ws_bytes = wsb;
    c->ws_b_bytes = wsb_b;
    const size_t act = (size_t)chunk_tokens * n * esz(dtype), wb = (size_t)n * m * esz(dtype);
    const size_t gb = (size_t)n * m * sizeof(float);
    bool ok = cudaStreamCreateWithFlags(&c->s_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&c->s_run, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&c->s_out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->w_ready, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < kBuf; ++i) {
        ok = cudaMalloc(&c->x[i], act) == cudaSuccess && cudaMalloc(&c->dy[i], act) == cudaSuccess &&
             cudaMalloc(&c->y[i], act) == cudaSuccess && cudaMalloc(&c->dx[i], act) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->in_ready[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->out_ready[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->out_done[i], cudaEventDisableTiming) == cudaSuccess;
    }
    ok = ok && cudaMalloc(&c->L, wb) == cudaSuccess && cudaMalloc(&c->R, wb) == cudaSuccess &&
         cudaMalloc(&c->dL, gb) == cudaSuccess && cudaMalloc(&c->dR, gb) == cudaSuccess &&
         cudaMalloc(&c->ws, wsb) == cudaSuccess && cudaMalloc(&c->ws_b, wsb_b) == cudaSuccess &&
         monarch_workspace_init(c->ws, wsb, c->s_run) == MONARCH_OK &&
         monarch_workspace_init(c->ws_b, wsb_b, c->s_run) == MONARCH_OK &&
         cudaStreamSynchronize(c->s_run) == cudaSuccess;
    if (!ok) {
        destroy(c);
        (void)cudaGetLastError();
        return MONARCH_ERR_CUDA;
    }
    *out = c;
    return MONARCH_OK;
}

int monarch_host_destroy(monarch_host_ctx *ctx)
{
    destroy(ctx);
    return MONARCH_OK;
}

int monarch_host_fwd(monarch_host_ctx *ctx, const void *x, const void *L, const void *R, void *y,
                     int64_t tokens)
{
    return run(ctx, x, nullptr, L, R, y, nullptr, nullptr, nullptr, tokens, false);
}

int monarch_host_fwd_bwd(monarch_host_ctx *ctx, const void *x, const void *dy, const void *L,
                         const void *R, void *y, void *dx, float *dL, float *dR, int64_t tokens)
{
    return run(ctx, x, dy, L, R, y, dx, dL, dR, tokens, true);
}

}  // extern "C"
