/*
 * ptq.h -- C ABI of the B200 (sm_100a) per-layer quantizer: sensitivity-ordered, row-parallel
 * quantization with one shared inverse Hessian (Sec. 4 of the paper).
 *
 * Data model (Sec. 3): W is [rows x cols] = d_row x d_col, X is [cols x n] = d_col x N, the layer
 * computes W X and the objective is ||W X - What X||^2 (Eq. 2).
 *
 * Rules common to every entry point
 *   - Every data pointer is a DEVICE pointer owned by the caller (unless a parameter says "host").
 *     The library allocates no device memory: scratch comes from the caller's workspace `ws`, whose
 *     minimum size is given by ptq_workspace_bytes().  Base pointers must be 16-byte aligned.
 *   - Matrices are row-major.  H, Hinv: float64 [cols x cols], full symmetric storage.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*).  The return value reports
 *     argument errors found on the host (nothing is launched then).  Conditions found on the device
 *     (not positive definite, non-finite input, bounded wait expired) are recorded in the caller's
 *     `status` word, int32[4] = {code, index, aux, 0}; the first error sticks, so the caller zeroes it
 *     before a sequence of calls and reads it after synchronising the stream.
 *   - Inputs are never modified; outputs are fully overwritten (H of ptq_hessian_accumulate is updated).
 *   - Results are deterministic: fixed reduction orders, no floating-point atomics.
 *   - Host-side state (SM count, kernel attributes) is kept per device and looked up with the caller's current
 *     device, so one process may drive several devices; calls may come from several host threads as long as calls
 *     that share a stream, a workspace or output buffers are ordered by the caller.
 *   - Size limits: ptq_quantize_layer (and its dynamic variant) takes rows <= 65535 and cols <= 65535, ptq_prepare_hinv
 *     cols <= 65535 (PTQ_ERR_UNSUPPORTED beyond).
 *   - No exceptions, no exit(), no stdout, no device trap, no unbounded device-side wait.
 */
#ifndef PTQ_H_
#define PTQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PTQ_OK = 0,
    PTQ_ERR_INVALID_ARG = 1,
    PTQ_ERR_ALIGNMENT = 2,
    PTQ_ERR_WORKSPACE = 3,
    PTQ_ERR_NOT_SPD = 4,     /* status[1] = failing pivot index */
    PTQ_ERR_NONFINITE = 5,
    PTQ_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired */
    PTQ_ERR_CUDA = 7,        /* a CUDA runtime call failed on the host */
    PTQ_ERR_UNSUPPORTED = 8,
    PTQ_ERR_STATIC_SCRATCH = 9 /* ptq_sensitivity_order_static: rows x cols beyond the built-in scratch array */
} ptq_status;

/* Damping (Implementation Details: a constant is added to the diagonal of H). */
typedef enum {
    PTQ_DAMP_REL_MEAN_DIAG = 0, /* lambda = damp * mean(diag H) */
    PTQ_DAMP_ABS = 1            /* lambda = damp (the paper's 0.1) */
} ptq_damp_mode;

/* Column score (Sec. 4.1 names the keys err / w / sensi; Sec. 4.2 step 2 sums them per column). */
typedef enum {
    PTQ_SCORE_QERR = 0,  /* Eq. 10: (w - quant(w))^2 / (2 [Hinv]_jj)   (default) */
    PTQ_SCORE_PRUNE = 1, /* Eq. 8 :  w^2 / (2 [Hinv]_jj) */
    PTQ_SCORE_ERR = 2,   /* (w - quant(w))^2 */
    PTQ_SCORE_W = 3,     /* w^2 */
    PTQ_SCORE_NONE = 4,  /* no sorting: identity order */
    /* Sec. 4.1 names each key in a descending ("des") and an ascending ("asc") variant.  Descending is the default
     * (and the method's); adding this flag to a mode sorts by S ascending.  Equal scores keep the lower column
     * index first in both directions. */
    PTQ_SCORE_ASCENDING = 16
} ptq_score_mode;

typedef enum {
    PTQ_CALL_HESSIAN_ACCUMULATE = 0,
    PTQ_CALL_PREPARE_HINV = 1,
    PTQ_CALL_SENSITIVITY_ORDER = 2,
    PTQ_CALL_QUANTIZE_LAYER = 3,
    PTQ_CALL_HESSIAN_ACCUMULATE_F64 = 4,
    PTQ_CALL_QUANTIZE_LAYER_DYNAMIC = 5,
    PTQ_CALL_QUANTIZE_LAYER_PER_ROW = 6
} ptq_call_id;

/* Minimum workspace, in bytes, for one call with these sizes (host function, no CUDA calls). */
size_t ptq_workspace_bytes(int call_id, int rows, int cols, int n);

/*
 * H += 2 * X X^T  (Sec. 3: the second derivative of Eq. 2 with respect to one row of W).
 *   H    [cols x cols] float64, in/out; the caller zeroes it before the first chunk of calibration columns
 *   X    [cols x n]    float32, row stride ldx >= n elements (vector loads are used when X is 16-byte aligned
 *                      and ldx is a multiple of 4)
 * The product is formed on the tensor cores from error-free integer slices of X, so H carries
 * float64-level accuracy (relative error about 1e-12 or better).
 */
int ptq_hessian_accumulate(double *H, const float *X, int cols, int n, int64_t ldx, void *ws, size_t ws_bytes,
                           int32_t *status, void *stream);

/*
 * The same accumulation for a convolutional layer, straight from the layer's input (Sec. 3: for a convolution d_col
 * is the number of weights of one filter, channels * kh * kw, and the columns of X are the input patches those
 * weights see).  With out_h = (height + 2 pad - kh) / stride + 1 (out_w alike), cols = channels * kh * kw and
 * n = batch * out_h * out_w:
 *     X[(c * kh + ki) * kw + kj][(b * out_h + oy) * out_w + ox] = act[b][c][oy * stride + ki - pad][ox * stride + kj - pad]
 * (zero outside the image), H += 2 X X^T.  The patches are never written out: the slicing pass reads act in place.
 *   H    [cols x cols] float64, in/out (row and column order: channel-major, then ki, then kj, the layout of a
 *        convolution weight [out_channels][channels][kh][kw] flattened per filter)
 *   act  [batch][channels][height][width] float32, contiguous
 * Workspace: ptq_workspace_bytes(PTQ_CALL_HESSIAN_ACCUMULATE, 0, cols, n).  Calling it once per calibration batch
 * accumulates over batches.  Sizes beyond cols = 2^20 or n = 2^30 return PTQ_ERR_UNSUPPORTED.
 */
int ptq_hessian_accumulate_conv(double *H, const float *act, int batch, int channels, int height, int width, int kh,
                                int kw, int stride, int pad, void *ws, size_t ws_bytes, int32_t *status, void *stream);

/* Same contract, computed with float64 FMAs (cross-check of the tensor-core path). */
int ptq_hessian_accumulate_f64(double *H, const float *X, int cols, int n, int64_t ldx, void *ws, size_t ws_bytes,
                               int32_t *status, void *stream);

/*
 * Hinv = (H + lambda I)^-1 by Cholesky factorisation and inversion of the factor (Sec. 5 item 1).
 *   H          [cols x cols] float64, const
 *   Hinv       [cols x cols] float64, out
 *   Hinv_diag  [cols] float64, out (the diagonal of Hinv, what the sensitivities need)
 *   lambda_out [1] float64, out (device)
 * A non-positive pivot sets status = {PTQ_ERR_NOT_SPD, pivot index}.
 */
int ptq_prepare_hinv(const double *H, int cols, int damp_mode, double damp, double *Hinv, double *Hinv_diag,
                     double *lambda_out, void *ws, size_t ws_bytes, int32_t *status, void *stream);

/*
 * Helper: per-row asymmetric min-max grid whose range always contains 0, from the original W
 * (Sec. 3, OBQ paragraph: a fixed grid of width Delta).  scale, zero: [rows] float32, out.
 * quant_i(w) = scale_i * (clamp(rint(w / scale_i) + zero_i, 0, 2^bits - 1) - zero_i), rint = ties to even.
 */
int ptq_minmax_grid(const float *W, int rows, int cols, int64_t ldw, int bits, float *scale, float *zero,
                    int32_t *status, void *stream);

/*
 * Sec. 4.2 steps 1-3: S_j = sum_i score(w_ij) from the original W and diag(Hinv); perm = columns by S descending
 * (ascending with PTQ_SCORE_ASCENDING added to score_mode), equal scores keep the lower column index first.
 * S [cols] float64 out, perm [cols] int32 out.
 */
int ptq_sensitivity_order(const float *W, int rows, int cols, int64_t ldw, const double *Hinv_diag, const float *scale,
                          const float *zero, int bits, int score_mode, double *S, int32_t *perm, void *ws,
                          size_t ws_bytes, int32_t *status, void *stream);

/*
 * ptq_sensitivity_order for callers that cannot hand the library any scratch memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above, with the same inputs, outputs and arithmetic.)
 *
 * Who needs it: code that runs where device allocation is off limits -- inside a region that must not call
 * cudaMalloc (a latency-critical serving loop, a process whose memory pool is owned and fully handed out by
 * another component, a plug-in that is given device pointers but no allocator) -- and that therefore cannot size
 * and provide the `ws` buffer the ordinary call asks for.  This entry point takes no workspace: the per-row-chunk
 * partial sums live in an array compiled into the library, PTQ_STATIC_SCRATCH_BYTES large.  Every device that loads
 * the library carries that array until the process exits, whether or not this function is ever called.
 *
 * Limits and rules
 *   - ceil(rows / 64) * cols * 8 bytes must not exceed PTQ_STATIC_SCRATCH_BYTES (e.g. 4096 x 11008 fits);
 *     larger problems return PTQ_ERR_STATIC_SCRATCH and launch nothing.
 *   - It never calls cudaMalloc, cudaFree or any allocating routine.  Every call looks up the array's device address
 *     (cudaGetSymbolAddress, with the caller's device current; nothing is remembered between calls, so the address
 *     is right after a cudaDeviceReset too).  The first such lookup on a device initialises the library's module
 *     there: make the first call on each device outside any stream capture.
 *   - All calls on one device share the one array, and it keeps whatever the previous call left there.  The
 *     kernels overwrite every element they later read, so no clearing is needed; but two calls that may run at
 *     the same time on the GPU (different streams, or different host threads) race on it: keep calls to this
 *     entry point ordered on one stream, or serialise them yourself.
 */
#define PTQ_STATIC_SCRATCH_BYTES (6u << 20)
int ptq_sensitivity_order_static(const float *W, int rows, int cols, int64_t ldw, const double *Hinv_diag,
                                 const float *scale, const float *zero, int bits, int score_mode, double *S,
                                 int32_t *perm, int32_t *status, void *stream);

/*
 * Sec. 4.2 steps 3-5: permute W and Hinv by perm, then quantize one column at a time, all rows in parallel;
 * after each column the remaining columns absorb the error (Eq. 11) and the shared inverse Hessian is
 * updated (Eq. 12).  The updates are applied in blocked form through the upper Cholesky factor of the
 * permuted inverse Hessian, whose row p equals row p of the Eq.-12-updated matrix divided by the square
 * root of its pivot.
 *   codes      [rows x cols] uint8, out, one code per byte, ORIGINAL column order
 *   What       [rows x cols] float32, out (may be NULL): scale_i * (code - zero_i)
 *   H_undamped [cols x cols] float64 and loss_out [1] float64 (device): loss = ||W X - What X||^2
 *              = 1/2 tr(dW H dW^T); pass NULL for either to skip
 */
int ptq_quantize_layer(const float *W, int rows, int cols, int64_t ldw, const double *Hinv, const int32_t *perm,
                       const float *scale, const float *zero, int bits, uint8_t *codes, float *What,
                       const double *H_undamped, double *loss_out, void *ws, size_t ws_bytes, int32_t *status,
                       void *stream);

/*
 * The column loop with dynamic re-ranking.  Sec. 5 writes the sort inside the per-column loop; read literally, the
 * columns still to be quantized are ranked again while the loop runs.  Every `block` columns the scores of the
 * REMAINING columns are recomputed from the current (compensated) weights and the diagonal of the current
 * (Eq.-12-updated) inverse Hessian, the remaining columns are sorted by them (keys, direction and tie rule of
 * ptq_sensitivity_order; ties by ORIGINAL column index) and the next `block` columns are quantized in that order
 * with Eq. 11 / Eq. 12.  block >= cols is ptq_sensitivity_order followed by ptq_quantize_layer.
 *   block      a multiple of 64, or >= cols (PTQ_ERR_UNSUPPORTED otherwise)
 *   order_out  [cols] int32, out: the sequence in which the columns were quantized
 *   other arguments as for ptq_quantize_layer (outputs in original column order); Hinv_diag is not needed
 * Workspace: ptq_workspace_bytes(PTQ_CALL_QUANTIZE_LAYER_DYNAMIC, rows, cols, 0).
 */
int ptq_quantize_layer_dynamic(const float *W, int rows, int cols, int64_t ldw, const double *Hinv, const float *scale,
                               const float *zero, int bits, int score_mode, int block, uint8_t *codes, float *What,
                               int32_t *order_out, const double *H_undamped, double *loss_out, void *ws,
                               size_t ws_bytes, int32_t *status, void *stream);

/*
 * The non-parallel arm of the paper's ablation (Sec. 4.2, the paragraph on the per-row inverse Hessians; Table 3's rows
 * without the parallel tick): every row ranks its own weights by their sensitivities (the keys of
 * ptq_sensitivity_order applied to that single row, Sec. 4.1) and is quantized in that order against its own copy of
 * the inverse Hessian -- what the shared-inverse-Hessian method avoids.  Cost rows * cols^3 / 3 and one cols x cols
 * matrix per row in flight, so only narrow layers are taken: cols <= 128 (PTQ_ERR_UNSUPPORTED beyond).
 *   perm_rows [rows x cols] int32, out: the order each row used
 *   other arguments as for ptq_quantize_layer; the diagonal of Hinv is read from Hinv itself
 * Workspace: ptq_workspace_bytes(PTQ_CALL_QUANTIZE_LAYER_PER_ROW, rows, cols, 0).
 */
int ptq_quantize_layer_per_row(const float *W, int rows, int cols, int64_t ldw, const double *Hinv, const float *scale,
                               const float *zero, int bits, int score_mode, uint8_t *codes, float *What,
                               int32_t *perm_rows, const double *H_undamped, double *loss_out, void *ws,
                               size_t ws_bytes, int32_t *status, void *stream);

/*
 * Sec. 4.2 step 3 alone: perm = the indices 0 .. cols-1 sorted by S descending (ascending != 0: ascending), equal
 * scores keep the lower index first.  For callers that form S themselves, e.g. by summing the per-shard scores of a
 * layer whose rows are spread over several GPUs (Sec. 4.2 step 2 is a sum over rows, so it splits over row shards).
 *   S [cols] float64, perm [cols] int32 out.  No workspace.
 */
int ptq_sort_scores(const double *S, int cols, int ascending, int32_t *perm, void *stream);

/*
 * C += alpha * A B^T for float64 operands, formed on the tensor cores from error-free int8 slices of the operands (the
 * way ptq_hessian_accumulate forms H), to float64 accuracy: the product behind the deferred part of Eq. 11,
 * W[:, later] -= E[:, block] U[block, later], exposed for cross-checks and for callers who want it on its own.
 *   C [m x n] float64, row stride ldc, in/out
 *   A [m x k] float64, row stride lda
 *   B: b_is_kn = 0: [n x k], row stride ldb;  b_is_kn = 1: the matrix is stored as [k x n] (so C += alpha A B), stride ldb
 *   k <= 16384 (PTQ_ERR_UNSUPPORTED beyond).  Rows of A / of B with wildly different magnitudes are fine (each has its
 *   own power-of-two scale); within a row, entries below 2^-54 of the row's largest magnitude are rounded away.
 * Workspace: ptq_gemm_nt_sliced_workspace_bytes(m, n, k).
 */
size_t ptq_gemm_nt_sliced_workspace_bytes(int m, int n, int k);
int ptq_gemm_nt_sliced(double *C, int64_t ldc, const double *A, int64_t lda, const double *B, int64_t ldb, int b_is_kn,
                       int m, int n, int k, double alpha, void *ws, size_t ws_bytes, int32_t *status, void *stream);

const char *ptq_status_string(int code);
int ptq_version(void);

/*
 * Self-test of the bounded device-side waits (instrumentation; the paper has no counterpart).  Launches a kernel that
 * calls the library's own wait routine on a target nothing will ever reach, with the given limit in SM clock cycles:
 *   which = 0 : the grid-wide barrier of the factorisation kernel (one CTA per SM), asked for one arrival too many
 *   which = 1 : the counter wait of the column sweep, on a counter that nobody raises
 * The wait must run out, the kernel records {PTQ_ERR_TIMEOUT, CTA index, 1 + which} in `status` and returns; the
 * context stays usable.  ws: at least 16 bytes of device scratch.  limit_cycles in [1, 4e9].
 */
int ptq_selftest_wait_timeout(int which, long long limit_cycles, void *ws, size_t ws_bytes, int32_t *status,
                              void *stream);

/*
 * Float64 throughput probe (instrumentation; the paper has no counterpart): launches one kernel of 4 CTAs x 256 threads
 * per SM in which every thread runs `iters` rounds of eight independent chains of float64 FMAs (kind 0) or of float64
 * tensor-core MMAs m8n8k4 (kind 1), and nothing else.  *flops_out (host) receives the floating-point operations of
 * that launch (FMA = 2); the caller times the launch on its stream.  sink: one device double (never written).
 */
int ptq_fp64_probe(int kind, int iters, double *sink, double *flops_out, void *stream);

/*
 * Launch accounting (instrumentation; the paper has no counterpart).  Host-side state of the calling process.
 *   ptq_kernel_count / ptq_kernel_name : the library's kernels, by id.
 *   ptq_launch_count(id)   : launches of kernel `id` since the library was loaded; id < 0 gives the total.
 *   ptq_profile_enable(on) : while on, every launch is bracketed by CUDA events on its stream (this perturbs
 *                            timing, so profile on passes that are not themselves being timed); each call clears
 *                            the records taken so far.
 *   ptq_profile_read(id, total_ms, launches) : host pointers; waits for the recorded events and sums the device
 *                            time of kernel `id` over the recorded launches.
 */
/* The two persistent cooperative kernels (factorisation, column sweep) launch one CTA per SM and occupy an SM each, so
 * two of them never share the GPU.  ptq_set_cta_limit(limit) makes the calls issued afterwards ON THE CURRENT DEVICE
 * launch at most `limit` CTAs (0: no limit, the default): a caller that runs independent layers on several streams sets
 * about sm_count / streams, so that their factorisations and sweeps run side by side (those of layers up to a few thousand
 * columns are bound by a dependency chain, not by the number of SMs).  Results do not depend on the limit.
 * Returns PTQ_ERR_INVALID_ARG for a negative limit. */
int ptq_set_cta_limit(int limit);

int ptq_kernel_count(void);
const char *ptq_kernel_name(int kernel_id);
long long ptq_launch_count(int kernel_id);
int ptq_profile_enable(int on);
int ptq_profile_read(int kernel_id, double *total_ms, long long *launches);

#ifdef __cplusplus
}
#endif
#endif /* PTQ_H_ */
