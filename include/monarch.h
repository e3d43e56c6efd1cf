/*
 * libmonarch - the Monarch matrix multiply on NVIDIA B200 (sm_100a), C ABI.
 *
 * A Monarch matrix (Dao et al., arXiv 2204.00595, Definition 3.1) of size
 * n x n, n = m*m, is  M = P L P^T R  with L and R block-diagonal (m blocks of
 * m x m each) and P the reshape(m,m)-transpose "stride" permutation.  The
 * calls below multiply a batch of token vectors by M, by M^T, form the
 * gradients of the blocks, and evaluate a Monarch feed-forward block.
 *
 * Conventions shared by every call (the monarch_host_* calls at the end of
 * this file take HOST pointers and own their device memory; they say so)
 * --------------------------------
 *  - All data pointers are DEVICE pointers owned by the caller, 16-byte
 *    aligned, dense and row-major.  Nothing is allocated, freed or retained
 *    by the library; outputs must not overlap inputs or the workspace.
 *  - x, y, dy, dx : [tokens][n]   (token-major; element k*m+i of a row is
 *    entry (k,i) of the m x m view of the vector used in Section 3.3).
 *  - L, R : [m][m][m] = [block][output row][input column]; i.e. R[k][j][i] and
 *    L[j][l][k] in the notation of Section 3.3 steps 1-2 and Algorithm 1.
 *  - b1, b2 : [n].
 *  - dtype MONARCH_F32 : every tensor is IEEE float32, fp32 arithmetic.
 *    dtype MONARCH_BF16: x, y, dy, dx, L, R, b1, b2 are bfloat16; products
 *    accumulate in fp32; on-chip intermediates (u, du, h) are rounded to
 *    bfloat16 once because they are tensor-core operands; dL, dR are float32.
 *  - n must equal m*m and m must be one of 16, 32, 64, 128; otherwise
 *    MONARCH_ERR_UNSUPPORTED.  tokens >= 0 (0 is a no-op that still defines
 *    dL/dR when accumulate == 0).
 *  - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it
 *    and return without synchronising.  Argument errors are reported by the
 *    return value before anything is enqueued.
 *  - `workspace` is caller-owned device scratch of at least
 *    monarch_workspace_bytes(op, ...) bytes, 256-byte aligned.  Its first
 *    MONARCH_STATUS_BYTES bytes hold a device status word that kernels set
 *    when one of their bounded waits runs out; zero it once with
 *    monarch_workspace_init and read it with monarch_last_device_status.
 *    Calls that overlap on the GPU must not share a workspace.
 *  - Weight gradients of the fused tensor-core kernels (bf16, m = 64; the
 *    general class) and of the staged tensor-core kernels (bf16, m = 32) are
 *    summed with fp32 reductions whose order across thread blocks is not
 *    fixed: dL, dR can differ in the last fp32 bits from run to run
 *    (monarch_set_deterministic switches m = 32 and m = 64 to a fixed order).  The bf16 m = 128 kernels (one thread block sums all tokens of a
 *    block, in a fixed order) and the CUDA-core family (MONARCH_IMPL_STAGED)
 *    give the same bits every run.
 *  - Return value: a monarch_status_t.  Nothing throws.
 */
#ifndef MONARCH_H_
#define MONARCH_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { MONARCH_F32 = 0, MONARCH_BF16 = 1 } monarch_dtype_t;

typedef enum {
    MONARCH_OK = 0,
    MONARCH_ERR_INVALID_ARG = 1, /* null / misaligned / overlapping pointer, n != m*m, bad enum */
    MONARCH_ERR_UNSUPPORTED = 2, /* m or dtype not built for this call */
    MONARCH_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or too small */
    MONARCH_ERR_CUDA = 4,        /* a CUDA runtime/driver call or a launch failed */
    MONARCH_ERR_TIMEOUT = 5      /* a kernel gave up on one of its bounded waits */
} monarch_status_t;

typedef enum {
    MONARCH_OP_FWD = 0,
    MONARCH_OP_BWD_DX = 1,
    MONARCH_OP_BWD_DW = 2,
    MONARCH_OP_MLP_FWD = 3,
    MONARCH_OP_BWD = 4, /* monarch_bwd: dx, dL and dR in one call */
    MONARCH_OP_MLP_BWD = 5,
    MONARCH_OP_CPLX = 6 /* monarch_cplx_fwd, either direction */
} monarch_op_t;

/* Which kernel family serves a call (process-wide; default AUTO). */
typedef enum {
    MONARCH_IMPL_AUTO = 0,   /* fused tensor-core kernels where built, else staged */
    MONARCH_IMPL_STAGED = 1, /* one block-diagonal stage per launch, CUDA-core FMA, any m */
    MONARCH_IMPL_FUSED = 2   /* fused tcgen05 kernels only; UNSUPPORTED where none exists */
} monarch_impl_t;

#define MONARCH_STATUS_BYTES 256

/* y = M x = P L P^T R x  (Definition 3.1; computed as Section 3.3 steps 1-3:
 * u[k][j] = sum_i R[k][j][i] x[k*m+i];  y[l*m+j] = sum_k L[j][l][k] u[k][j]). */
int monarch_fwd(const void *x, const void *L, const void *R, void *y,
                int64_t tokens, int32_t n, int32_t m, int dtype,
                void *workspace, size_t workspace_bytes, void *stream);

/* dx = M^T dy = R^T P L^T P dy, the adjoint of steps 1-3 (the paper trains by
 * automatic differentiation, Section 4):
 * du[k][j] = sum_l L[j][l][k] dy[l*m+j];  dx[k*m+i] = sum_j R[k][j][i] du[k][j]. */
int monarch_bwd_dx(const void *dy, const void *L, const void *R, void *dx,
                   int64_t tokens, int32_t n, int32_t m, int dtype,
                   void *workspace, size_t workspace_bytes, void *stream);

/* Gradients of the blocks for f = <dy, M x> summed over tokens:
 * dL[j][l][k] = sum_t dy[t][l*m+j] u[t][k][j],  dR[k][j][i] = sum_t du[t][k][j] x[t][k*m+i],
 * with u, du as above (recomputed inside).  dL, dR are float32 [m][m][m] in
 * both dtypes; accumulate == 0 overwrites them, 1 adds to their contents. */
int monarch_bwd_dw(const void *x, const void *dy, const void *L, const void *R,
                   float *dL, float *dR, int accumulate,
                   int64_t tokens, int32_t n, int32_t m, int dtype,
                   void *workspace, size_t workspace_bytes, void *stream);

/* The whole backward pass in one call: dx as in monarch_bwd_dx and dL, dR as in
 * monarch_bwd_dw, sharing du (and reading dy once).  `fwd_workspace` is either
 * null or the workspace that monarch_fwd used for the SAME x, L, R, tokens, n,
 * m, dtype, untouched since that call returned its work to the stream: kernel
 * families that keep u = P^T R x there in a layout they can read back use it
 * instead of recomputing u (as an autograd function saves its intermediate);
 * the others ignore it.  The caller vouches for its contents; a stale buffer
 * gives a wrong dL, not an error.  `workspace` (monarch_workspace_bytes with
 * MONARCH_OP_BWD) must not be the same buffer as `fwd_workspace`. */
int monarch_bwd(const void *x, const void *dy, const void *L, const void *R,
                const void *fwd_workspace, void *dx, float *dL, float *dR, int accumulate,
                int64_t tokens, int32_t n, int32_t m, int dtype,
                void *workspace, size_t workspace_bytes, void *stream);

/* Monarch feed-forward block (Section 4: the FFN weights replaced by Monarch
 * matrices):  y = M2 GELU(M1 x + b1) + b2,  M1 = P L1 P^T R1, M2 = P L2 P^T R2,
 * GELU(a) = a/2 (1 + erf(a / sqrt 2)). */
int monarch_mlp_fwd(const void *x, const void *L1, const void *R1, const void *b1,
                    const void *L2, const void *R2, const void *b2, void *y,
                    int64_t tokens, int32_t n, int32_t m, int dtype,
                    void *workspace, size_t workspace_bytes, void *stream);

/* Gradients of f = <dy, y> for the feed-forward block above (Section 4 trains
 * it by automatic differentiation; this is that chain rule):
 *   a = M1 x + b1,  h = GELU(a)                       (recomputed inside)
 *   dh = M2^T dy,   dL2, dR2 = block gradients of M2 with input h,   db2 = sum_t dy[t]
 *   da = dh * GELU'(a),  GELU'(a) = (1 + erf(a/sqrt 2))/2 + a exp(-a^2/2)/sqrt(2 pi)
 *   dx = M1^T da,   dL1, dR1 = block gradients of M1 with input x,   db1 = sum_t da[t]
 * x, dy, dx: [tokens][n] in the storage dtype; b1: [n] storage dtype (b2 does
 * not enter the gradients).  dL1, dR1, dL2, dR2: float32 [m][m][m]; db1, db2:
 * float32 [n]; accumulate == 0 overwrites all six, 1 adds to their contents.
 * a, h and da are rounded to the storage dtype once each (they are tensor-core
 * operands).  The sums over tokens use atomic adds: their order, hence the
 * last bits, may vary from run to run.  Workspace: monarch_workspace_bytes
 * with MONARCH_OP_MLP_BWD. */
int monarch_mlp_bwd(const void *x, const void *dy, const void *L1, const void *R1, const void *b1,
                    const void *L2, const void *R2, void *dx,
                    float *dL1, float *dR1, float *db1, float *dL2, float *dR2, float *db2,
                    int accumulate, int64_t tokens, int32_t n, int32_t m, int dtype,
                    void *workspace, size_t workspace_bytes, void *stream);

/* General (rectangular) Monarch multiply of the appendix "General Monarch
 * Matrix Parametrization":  y = L R x  with
 *   R = diag(R_0 .. R_{q-1}), R_k of size b x b1   (n1 = q*b1 inputs, n2 = q*b),
 *   L of size n3 x n2 (n3 = r*b): an r x q grid of b x b diagonal blocks S_{l,k}
 * (the case b2 = b3 = b of the rectangular definition, the one its
 * block-diagonalisation theorem covers; q = b1 = b = r = m is Definition 3.1).
 * Steps:  u[t][k*b + j] = sum_i R[k][j][i] x[t][k*b1 + i]
 *         y[t][l*b + j] = sum_k L[j][l][k] u[t][k*b + j].
 * x: [tokens][q*b1], y: [tokens][r*b], row-major, storage dtype;
 * R: [q][b][b1];  L: [b][r][q] with L[j][l][k] = S_{l,k}[j][j], i.e. the b
 * blocks (r x q) of the block-diagonal form P L P^T of that theorem.
 * u is rounded to the storage dtype once (fp32 accumulation throughout).
 * All four sizes must be in [1, 16384] and every row (q*b1, q*b, r*b) at most
 * 2^24 elements; MONARCH_ERR_UNSUPPORTED otherwise.  Workspace:
 * monarch_rect_workspace_bytes (0 for invalid arguments). */
int monarch_rect_fwd(const void *x, const void *L, const void *R, void *y, int64_t tokens,
                     int32_t q, int32_t b1, int32_t b, int32_t r, int dtype,
                     void *workspace, size_t workspace_bytes, void *stream);
size_t monarch_rect_workspace_bytes(int64_t tokens, int32_t q, int32_t b1, int32_t b, int32_t r,
                                    int dtype);

/* Gradients of f = <dy, L R x> for the general class (adjoints of the two steps
 * above; the paper trains these layers by automatic differentiation):
 *   du[t][k*b + j]  = sum_l L[j][l][k] dy[t][l*b + j]
 *   dx[t][k*b1 + i] = sum_j R[k][j][i] du[t][k*b + j]
 *   dL[j][l][k] = sum_t dy[t][l*b + j] u[t][k*b + j],  dR[k][j][i] = sum_t du[t][k*b + j] x[t][k*b1 + i]
 * `fwd_workspace` is null (u is recomputed inside) or the workspace that
 * monarch_rect_fwd used for the SAME x, R and sizes, untouched since: u is then
 * read from there (the caller vouches for its contents, as for monarch_bwd).
 * x, dx: [tokens][q*b1]; dy: [tokens][r*b]; dL:
 * float32 [b][r][q]; dR: float32 [q][b][b1]; accumulate == 0 overwrites the two
 * weight gradients, 1 adds to them.  u and du are rounded to the storage dtype
 * once; the sums over tokens use atomic adds (last bits may vary run to run).
 * Workspace: monarch_rect_bwd_workspace_bytes. */
int monarch_rect_bwd(const void *x, const void *dy, const void *L, const void *R,
                     const void *fwd_workspace,
                     void *dx, float *dL, float *dR, int accumulate, int64_t tokens,
                     int32_t q, int32_t b1, int32_t b, int32_t r, int dtype,
                     void *workspace, size_t workspace_bytes, void *stream);
size_t monarch_rect_bwd_workspace_bytes(int64_t tokens, int32_t q, int32_t b1, int32_t b,
                                        int32_t r, int dtype);

/* The rectangular class with WRAPPED-DIAGONAL blocks (appendix "General Monarch
 * Matrix Parametrization", rectangular definition with b2 != b3):  y = L R x,
 *   R = diag(R_0 .. R_{q-1}), R_k of size b2 x b1  (n1 = q*b1 inputs, n2 = q*b2),
 *   L of size n3 x n2 (n3 = r*b3): an r x q grid of blocks S_{l,k} of size b3 x b2,
 *   each a wrapped diagonal with max(b2, b3) entries: for b2 <= b3 row i0 has its
 *   one non-zero in column i0 mod b2; for b2 > b3 column j0 has its one non-zero
 *   in row j0 mod b3 (the definition applied to the transpose).
 * Stored entry e of a block sits at (i0, j0) = (e, e mod b2) if b2 <= b3, else
 * (e mod b3, e).  Steps:
 *   u[t][k*b2 + j] = sum_i R[k][j][i] x[t][k*b1 + i]
 *   y[t][l*b3 + i0(e)] += L[l][k][e] u[t][k*b2 + j0(e)]    over all k and e.
 * x: [tokens][q*b1], y: [tokens][r*b3], storage dtype; R: [q][b2][b1];
 * L: [r][q][max(b2, b3)].  b2 == b3 is monarch_rect_fwd with L[l][k][j] there
 * stored as L[j][l][k].  Where one of b2, b3 divides the other the product is a
 * diagonal-block product of other sizes and runs on those kernels after the
 * weights are re-labelled in the workspace; other sizes run on plain CUDA-core
 * kernels.  u is rounded to the storage dtype once.  Size limits and errors as
 * for monarch_rect_fwd.  The backward call returns dx, dL (float32, laid out like
 * L) and dR (float32 [q][b2][b1]) of f = <dy, L R x>; accumulate == 0 overwrites
 * the two weight gradients, 1 adds to them; the sums over tokens use atomic adds.
 * Workspaces: monarch_rectw_workspace_bytes, monarch_rectw_bwd_workspace_bytes
 * (0 for invalid arguments). */
int monarch_rectw_fwd(const void *x, const void *L, const void *R, void *y, int64_t tokens,
                      int32_t q, int32_t b1, int32_t b2, int32_t b3, int32_t r, int dtype,
                      void *workspace, size_t workspace_bytes, void *stream);
size_t monarch_rectw_workspace_bytes(int64_t tokens, int32_t q, int32_t b1, int32_t b2, int32_t b3,
                                     int32_t r, int dtype);
int monarch_rectw_bwd(const void *x, const void *dy, const void *L, const void *R,
                      void *dx, float *dL, float *dR, int accumulate, int64_t tokens,
                      int32_t q, int32_t b1, int32_t b2, int32_t b3, int32_t r, int dtype,
                      void *workspace, size_t workspace_bytes, void *stream);
size_t monarch_rectw_bwd_workspace_bytes(int64_t tokens, int32_t q, int32_t b1, int32_t b2,
                                         int32_t b3, int32_t r, int dtype);

/* Complex Monarch multiply (Section 3.2: the DFT and the MM* products need
 * complex factors):  y = M x  (adjoint == 0)  or  y = M^H x  (adjoint == 1),
 * M = P L P^T R with complex blocks, M^H = R^H P L^H P.  An MM* product
 * M1 M2^H x is two calls.  Complex tensors are PLANAR in the storage dtype:
 * x, y: [2][tokens][n] (real plane, then imaginary plane); L, R: [2][m][m][m].
 * The call runs four real Monarch multiplies over both planes at once
 * (M(Lr,Rr), M(Li,Ri), M(Lr,Ri), M(Li,Rr) applied to [xr; xi]) and combines
 * them:  Re M = M(Lr,Rr) - M(Li,Ri),  Im M = M(Lr,Ri) + M(Li,Rr); each of the
 * four results is rounded to the storage dtype before the combination.
 * Workspace: monarch_workspace_bytes with MONARCH_OP_CPLX. */
int monarch_cplx_fwd(const void *x, const void *L, const void *R, void *y, int adjoint,
                     int64_t tokens, int32_t n, int32_t m, int dtype,
                     void *workspace, size_t workspace_bytes, void *stream);

/* Dense materialisation by the entry formula, Eq. (2):
 *   M[l*m+j][k*m+i] = L[j][l][k] * R[k][j][i],   M: [n][n] row-major, storage dtype
 * (the product is formed in fp32 and rounded once). */
int monarch_dense(const void *L, const void *R, void *M, int32_t n, int32_t m, int dtype,
                  void *stream);

/* Projection of a dense matrix onto the Monarch class, Algorithm 1: with
 * A~[l][j][k][i] = A[l*m+j][k*m+i], every m x m slice A~[:, j, k, :] is replaced
 * by its best rank-1 approximation sigma_1 u_1 v_1^T (Theorem 1: this minimises
 * ||A - M||_F over Monarch M), stored as L[j][:, k] = sqrt(sigma_1) u_1 and
 * R[k][j][:] = sqrt(sigma_1) v_1.  The paper fixes only the product u v^T; the
 * sign of the pair is arbitrary, and where sigma_1 = sigma_2 the slice's
 * approximation itself is not unique.  A: [n][n] row-major; L, R: [m][m][m];
 * all in the storage dtype, arithmetic in fp32 (one-sided Jacobi per slice).
 * `rotation_count` is null or a device counter to which the number of plane
 * rotations performed is added (for FLOP accounting). */
int monarch_project(const void *A, void *L, void *R, int32_t n, int32_t m, int dtype,
                    unsigned long long *rotation_count, void *stream);

/* Bytes of workspace `op` (a monarch_op_t) needs for these sizes under the
 * current implementation choice; always >= MONARCH_STATUS_BYTES.  Returns 0
 * for invalid or unsupported arguments. */
size_t monarch_workspace_bytes(int op, int64_t tokens, int32_t n, int32_t m, int dtype);

/* Zero the status word and the tile counters that follow it (enqueued on
 * `stream`); call once before the first use of a workspace. */
int monarch_workspace_init(void *workspace, size_t workspace_bytes, void *stream);

/* Synchronise `stream`, read and clear the status word: MONARCH_OK, or
 * MONARCH_ERR_TIMEOUT if a kernel abandoned a bounded wait since the last
 * query (its outputs are then undefined, and the tile counters in the
 * workspace may be left non-zero: call monarch_workspace_init again before
 * reusing it), or MONARCH_ERR_CUDA. */
int monarch_last_device_status(void *workspace, void *stream);

/* Test aids for the bounded waits (the paper has no counterpart; they exist so that the
 * time-out path can be exercised without faulting or hanging a GPU).
 * monarch_debug_set_wait_limit: kernels that use `workspace` from now on give up a wait after
 * `microseconds` instead of about one second (0 restores the default; monarch_workspace_init
 * also does).  Enqueued on `stream`.
 * monarch_debug_skip_load: host-side fault injection.  The next m = 128 forward call leaves out
 * one operand load of its last step (item = tile * 128 + output row block; -1 cancels), so the
 * thread block that owns the item waits for data that never arrives, gives up after the wait
 * limit, records MONARCH_ERR_TIMEOUT in the status word and returns; its outputs are undefined.
 * Nothing faults and no wait is unbounded. */
int monarch_debug_set_wait_limit(void *workspace, unsigned int microseconds, void *stream);
int monarch_debug_skip_load(int64_t item);

/* Select the kernel family for later calls (a monarch_impl_t).  Not
 * thread-safe against concurrent calls. Returns the previous value, or -1. */
int monarch_set_impl(int impl);

/* Summation order of the weight gradients dL[j][l][k] = sum_t dy[t][l*m+j] u[t][k][j]
 * and dR[k][j][i] = sum_t du[t][k][j] x[t][k*m+i] (the adjoints of Section 3.3,
 * steps 1-2) in the bf16 kernels that split the tokens over thread blocks: m = 64
 * (fused family) and m = 32 (staged tensor-core family), behind monarch_bwd and
 * monarch_bwd_dw.  on != 0: every thread block writes the partial sums of its
 * (fixed) share of the token tiles to the workspace and a second small launch adds
 * them in a fixed order - the same bits on every run, accumulate honoured by that
 * launch; monarch_workspace_bytes for these two operations then reports 32 MiB
 * more, and at m = 64 a device on which the one-launch backward cannot run gets
 * MONARCH_ERR_UNSUPPORTED instead of the multi-launch form.  on == 0 (default):
 * partial sums are added with fp32 atomics in whatever order they arrive.  Other
 * sizes and dtypes already sum in a fixed order (bf16 m = 128, every fp32 call) or
 * are not affected (the feed-forward block and the general class keep their
 * atomics).  Process-wide, affects later calls and later workspace-size queries;
 * not thread-safe against concurrent calls.  Returns the previous setting. */
int monarch_set_deterministic(int on);

/* Name of the kernel family the next call with these arguments would use
 * ("staged-simt", "fused-simt", "staged-tcgen05", "fused-tcgen05"; "unsupported").  Static storage. */
const char *monarch_impl_name(int op, int32_t m, int dtype);

/* Number of kernel launches the library has enqueued since load (for
 * benchmarks that report their launch count). */
uint64_t monarch_launch_count(void);

const char *monarch_status_string(int status);

/* ---- Host-buffer calls ---------------------------------------------------
 * For callers whose tensors live in HOST memory.  A context owns the device
 * buffers (three token chunks of x, dy, y, dx, the weights, dL/dR and a
 * workspace) and three streams; a call uploads chunk c+1, runs the device
 * entry points above on chunk c and downloads chunk c-1 concurrently, and
 * returns after everything has arrived.  The arithmetic is exactly that of
 * monarch_fwd / monarch_bwd_dx / monarch_bwd_dw (Section 3.3 steps 1-3 and
 * their adjoints); the paper has no counterpart of the staging itself.
 *
 * All data pointers of these calls are HOST pointers owned by the caller
 * (page-locked memory lets the copies overlap; pageable memory is accepted
 * and serialises them), layouts and dtypes as above.  The calls block until
 * the outputs are complete and are not re-entrant on one context.
 *
 * monarch_host_create: max_tokens bounds later calls; chunk_tokens is the
 * staging granularity (a multiple of 64; 0 picks max_tokens / 8 rounded up to
 * 64 and clamped to [256, 2048], so that uploads and downloads of different
 * chunks overlap for most of a call).  Allocates
 * device memory with cudaMalloc on the current device; MONARCH_ERR_CUDA if
 * that fails, MONARCH_ERR_UNSUPPORTED / MONARCH_ERR_INVALID_ARG for bad
 * shapes.  monarch_host_destroy frees everything (null is a no-op). */
typedef struct monarch_host_ctx monarch_host_ctx;
int monarch_host_create(monarch_host_ctx **out, int64_t max_tokens, int32_t n, int32_t m,
                        int dtype, int64_t chunk_tokens);
int monarch_host_destroy(monarch_host_ctx *ctx);

/* y = M x on host buffers ([tokens][n] each; L, R [m][m][m]). */
int monarch_host_fwd(monarch_host_ctx *ctx, const void *x, const void *L, const void *R,
                     void *y, int64_t tokens);

/* One training step on host buffers: y = M x, dx = M^T dy, and dL, dR (float32,
 * overwritten) summed over all tokens.  Returns MONARCH_ERR_TIMEOUT if a
 * kernel reported an abandoned wait. */
int monarch_host_fwd_bwd(monarch_host_ctx *ctx, const void *x, const void *dy, const void *L,
                         const void *R, void *y, void *dx, float *dL, float *dR,
                         int64_t tokens);

/* Forward pass y = M x for callers that cannot allocate device memory - code running where
 * cudaMalloc is off limits (a real-time or serving loop whose device memory was fixed at
 * start-up, a plug-in under a host framework that owns the whole device heap, a process
 * whose memory budget is already spent) and that has no spare buffer to lend as a workspace.
 * The paper has no counterpart; this is a convenience of this library.
 *
 * Same arguments, layouts and results as monarch_fwd, minus the workspace: the
 * intermediate between the two stages is kept in an array built into the library
 * (MONARCH_NOALLOC_SCRATCH_BYTES, resident on every GPU that loads the library until the
 * process exits).  The call allocates and frees nothing.
 *
 *  - Limit: tokens * n * sizeof(element) must not exceed MONARCH_NOALLOC_SCRATCH_BYTES
 *    (e.g. 1024 tokens of n = 4096 in bf16); larger problems return
 *    MONARCH_ERR_WORKSPACE and enqueue nothing - split the batch or use monarch_fwd.
 *  - The first call on each device looks up the device address of the built-in array
 *    (with that device current).  Make that first call before starting any stream capture.
 *  - All calls share the one array and it keeps the previous call's contents.  Nothing in
 *    it has to start at zero (each call overwrites what it later reads), but two calls
 *    that may run at the same time on one GPU - different streams, or different host
 *    threads - race on it: serialise them on one stream.
 *  - Served by the staged kernel family regardless of monarch_set_impl.
 */
#define MONARCH_NOALLOC_SCRATCH_BYTES (8u << 20)
int monarch_fwd_noalloc(const void *x, const void *L, const void *R, void *y,
                        int64_t tokens, int32_t n, int32_t m, int dtype, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MONARCH_H_ */
