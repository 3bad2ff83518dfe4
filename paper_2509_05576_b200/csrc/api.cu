// C-ABI entry points (see include/ptq.h): argument checks, workspace carving, kernel sequencing.
#include "common.cuh"
#include "dgemm.cuh"
#include "chol.cuh"
#include "order.cuh"
#include "colloop.cuh"
#include "gram.cuh"
#include "dynamic.cuh"
#include "perrow.cuh"
#include "i8gemm.cuh"
#include "cholpanel.cuh"

using namespace ptq;

namespace {

__global__ void convert_f32_f64_kernel(const float* __restrict__ X, int rows, int n, int64_t ldx,
                                       double* __restrict__ Xd) {
    const int i = blockIdx.y;
    for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < n; k += gridDim.x * blockDim.x)
        Xd[(int64_t)i * n + k] = (double)X[(int64_t)i * ldx + k];
}

inline int grid_x_for(int n, int threads) {
    int g = cdiv(n, threads);
    return g < 1 ? 1 : (g > 1024 ? 1024 : g);
}

// The loss product is cut along k into as many slices as it takes to put about two CTAs on every SM.
constexpr int kMaxGridY = 65535;
constexpr int kSuperBlock = 1024;         // columns swept per launch on tall, wide layers
constexpr int kSuperBlockMinRows = 2048;
constexpr int kSlicedMinCols = 3072;      // from here on the large float64 products run on the int8 tensor path
constexpr int kLossMaxSplit = 8;
int loss_ksplit(int rows, int cols) {
    const long ctas = (long)cdiv(rows, 64) * ((cdiv(cols, 64) + 1) / 2);
    const long want = (2 * 148 + ctas - 1) / ctas;
    return (int)(want < 1 ? 1 : (want > kLossMaxSplit ? kLossMaxSplit : want));
}
size_t loss_partials_count(int rows, int cols) {
    return (size_t)kLossMaxSplit * cdiv(rows, 64) * cdiv(cols, 64);
}

// Built-in scratch of ptq_sensitivity_order_static: lives in every device that loads the library, until exit.
constexpr size_t kStaticScratchDoubles = PTQ_STATIC_SCRATCH_BYTES / sizeof(double);
static __device__ __align__(256) double g_static_score_scratch[kStaticScratchDoubles];

// Device address of the array on the current device.  In host code the symbol's name is only a handle, so the
// address is asked of the runtime, with the caller's device current, on every call: the lookup is cheap after the
// first one, and an address remembered across a cudaDeviceReset or under another context would be stale.
int static_scratch_address(double** out) {
    double* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_static_score_scratch) != cudaSuccess || !p) {
        cudaGetLastError();
        return PTQ_ERR_CUDA;
    }
    *out = p;
    return PTQ_OK;
}

// Scores and order (Sec. 4.2 steps 1-3) with the per-row-chunk partial sums in `partial`.
int order_launch(const float* W, int rows, int cols, int64_t ldw, const double* Hinv_diag, const float* scale,
                 const float* zero, int bits, int mode, int ascending, double* S, int32_t* perm, double* partial,
                 int32_t* status, cudaStream_t stream) {
    const int chunks = cdiv(rows, kScoreRowChunk);
    if (chunks > 65535) return PTQ_ERR_UNSUPPORTED;
    if (mode != PTQ_SCORE_NONE) {
        Launch l(K_SCORE_PARTIAL, stream);
        score_partial_kernel<float><<<dim3(cdiv(cols, kScoreCols), chunks), 256, 0, stream>>>(W, rows, cols, ldw, scale,
                                                                                            zero, bits, mode, partial);
    }
    { Launch l(K_SCORE_FINAL, stream); score_final_kernel<<<cdiv(cols, 128), 128, 0, stream>>>(partial, chunks, cols, Hinv_diag, mode, S, status); }
    { Launch l(K_RANK_SORT, stream); rank_sort_kernel<<<cdiv(cols, kRankCols), 256, 0, stream>>>(S, cols, ascending, perm); }
    return launch_status();
}

int order_args_check(const float* W, int rows, int cols, int64_t ldw, const double* Hinv_diag, const float* scale,
                     const float* zero, int bits, int score_mode, const double* S, const int32_t* perm) {
    if (!W || !S || !perm || rows < 1 || cols < 1 || ldw < cols || bits < 2 || bits > 8) return PTQ_ERR_INVALID_ARG;
    if (score_mode & ~(PTQ_SCORE_ASCENDING | 7)) return PTQ_ERR_INVALID_ARG;
    const int mode = score_mode & ~PTQ_SCORE_ASCENDING;
    if (mode < PTQ_SCORE_QERR || mode > PTQ_SCORE_NONE) return PTQ_ERR_INVALID_ARG;
    if ((mode == PTQ_SCORE_QERR || mode == PTQ_SCORE_PRUNE) && !Hinv_diag) return PTQ_ERR_INVALID_ARG;
    if ((mode == PTQ_SCORE_QERR || mode == PTQ_SCORE_ERR) && (!scale || !zero)) return PTQ_ERR_INVALID_ARG;
    return PTQ_OK;
}

// Self-test kernels: they call the very wait routines of the factorisation and of the sweep on a target that nothing
// will ever reach, so that the wait must run out, report PTQ_ERR_TIMEOUT and return.
__global__ void __launch_bounds__(kCholThreads) selftest_barrier_kernel(unsigned* bar, int32_t* status, long long spin_limit) {
    __shared__ int s_flag;
    const bool ok = grid_barrier(bar, gridDim.x + 1u, &s_flag, spin_limit);      // one arrival more than the grid has
    if (!ok && threadIdx.x == 0) report(status, PTQ_ERR_TIMEOUT, blockIdx.x, 1);
}
__global__ void selftest_counter_kernel(unsigned* words, int32_t* status, long long spin_limit) {
    if (threadIdx.x == 0 && !bounded_counter_wait(&words[0], 1u, &words[1], spin_limit))
        report(status, PTQ_ERR_TIMEOUT, blockIdx.x, 2);
}

// Float64 throughput probes: eight independent chains per thread, nothing but the arithmetic instruction in the loop.
constexpr int kProbeThreads = 256, kProbeCtasPerSm = 4, kProbeChains = 8;
__global__ void __launch_bounds__(kProbeThreads) fp64_probe_fma_kernel(int iters, double* sink) {
    double acc[kProbeChains];
    const double a = 1.0 + 1e-9 * threadIdx.x, b = 1e-12 * (blockIdx.x + 1);
#pragma unroll
    for (int c = 0; c < kProbeChains; ++c) acc[c] = (double)c;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int c = 0; c < kProbeChains; ++c) acc[c] = fma(acc[c], a, b);
    }
    double s = 0.0;
#pragma unroll
    for (int c = 0; c < kProbeChains; ++c) s += acc[c];
    if (s == 123.456) sink[0] = s;          // never true: keeps the loop alive without a store per thread
}
__global__ void __launch_bounds__(kProbeThreads) fp64_probe_mma_kernel(int iters, double* sink) {
    double acc[kProbeChains][2];
    const double a = 1.0 + 1e-9 * threadIdx.x, b = 1e-3 * ((threadIdx.x & 3) + 1);
#pragma unroll
    for (int c = 0; c < kProbeChains; ++c) acc[c][0] = acc[c][1] = 1e-12 * c;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int c = 0; c < kProbeChains; ++c) dmma_884(acc[c][0], acc[c][1], a, b);
    }
    double s = 0.0;
#pragma unroll
    for (int c = 0; c < kProbeChains; ++c) s += acc[c][0] + acc[c][1];
    if (s == 123.456) sink[0] = s;
}

}  // namespace

extern "C" {

int ptq_version(void) { return 1; }

int ptq_kernel_count(void) { return K_COUNT; }

const char* ptq_kernel_name(int kernel_id) { return kernel_name(kernel_id); }

long long ptq_launch_count(int kernel_id) {
    const Profiler& p = profiler();
    if (kernel_id >= 0 && kernel_id < K_COUNT) return p.launches[kernel_id];
    long long total = 0;
    for (int k = 0; k < K_COUNT; ++k) total += p.launches[k];
    return total;
}

int ptq_set_cta_limit(int limit) {
    if (limit < 0) return PTQ_ERR_INVALID_ARG;
    DeviceState* dev = nullptr;
    const int st = current_device_state(&dev);
    if (st) return st;
    std::lock_guard<std::mutex> lock(host_state_mutex());
    dev->cta_limit = limit;
    return PTQ_OK;
}

int ptq_profile_enable(int on) {
    Profiler& p = profiler();
    p.clear();
    p.on = on != 0;
    return PTQ_OK;
}

int ptq_profile_read(int kernel_id, double* total_ms, long long* launches) {
    Profiler& p = profiler();
    if (kernel_id < 0 || kernel_id >= K_COUNT || !total_ms || !launches) return PTQ_ERR_INVALID_ARG;
    double ms = 0.0;
    long long cnt = 0;
    for (const auto& r : p.recs) {
        if (r.id != kernel_id) continue;
        if (cudaEventSynchronize(r.b) != cudaSuccess) return PTQ_ERR_CUDA;
        float t = 0.f;
        if (cudaEventElapsedTime(&t, r.a, r.b) != cudaSuccess) return PTQ_ERR_CUDA;
        ms += (double)t;
        ++cnt;
    }
    *total_ms = ms;
    *launches = cnt;
    return PTQ_OK;
}

const char* ptq_status_string(int code) {
    switch (code) {
        case PTQ_OK: return "ok";
        case PTQ_ERR_INVALID_ARG: return "invalid argument";
        case PTQ_ERR_ALIGNMENT: return "pointer or leading dimension not aligned";
        case PTQ_ERR_WORKSPACE: return "workspace too small";
        case PTQ_ERR_NOT_SPD: return "matrix not positive definite";
        case PTQ_ERR_NONFINITE: return "non-finite value";
        case PTQ_ERR_TIMEOUT: return "bounded device wait expired";
        case PTQ_ERR_CUDA: return "CUDA runtime error";
        case PTQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case PTQ_ERR_STATIC_SCRATCH: return "problem too large for the built-in scratch array";
        default: return "unknown status";
    }
}

size_t ptq_workspace_bytes(int call_id, int rows, int cols, int n) {
    if (cols < 1) return 0;
    const size_t c = (size_t)cols;
    size_t total = 0;
    auto add = [&](size_t bytes) { total += align_up(bytes); };
    switch (call_id) {
        case PTQ_CALL_HESSIAN_ACCUMULATE:
            if (n < 1) return 0;
            return gram_workspace_bytes(cols, n);
        case PTQ_CALL_HESSIAN_ACCUMULATE_F64:
            if (n < 1) return 0;
            add(c * (size_t)n * sizeof(double));
            break;
        case PTQ_CALL_PREPARE_HINV:
            add(c * c * sizeof(double));
            add(c * c * sizeof(double));
            add(2 * sizeof(unsigned));                      // grid barrier of the factorisation kernel
            add(chol_scratch_doubles(cols) * sizeof(double));
            add(chol_panel_workspace_bytes(cols));          // operand slices of the panel updates (large matrices)
            break;
        case PTQ_CALL_SENSITIVITY_ORDER:
            if (rows < 1) return 0;
            add((size_t)cdiv(rows, kScoreRowChunk) * c * sizeof(double));
            break;
        case PTQ_CALL_QUANTIZE_LAYER:
            if (rows < 1) return 0;
            add(c * c * sizeof(double));                    // permuted inverse Hessian -> its factor U
            add((size_t)rows * c * sizeof(double));         // permuted W (float64), later dW
            add((size_t)rows * c * sizeof(double));         // scaled errors E
            add((size_t)rows * c);                          // codes in permuted order
            add(c * sizeof(int32_t));                       // flags
            add(c * sizeof(int32_t));                       // inverse permutation
            add(loss_partials_count(rows, cols) * sizeof(double));
            add(2 * sizeof(unsigned));                      // grid barrier of the factorisation kernel
            add(((size_t)cdiv(rows, kSweepRows) + 1) * sizeof(unsigned));   // per-row-group progress counters of the sweep
            add(chol_scratch_doubles(cols) * sizeof(double));
            if (rows >= kSuperBlockMinRows && cols >= 4 * kSuperBlock)
                add(i8gemm_workspace_bytes(rows, cols, kSuperBlock));   // slices of E[:, sb] and U[sb, later]
            add(chol_panel_workspace_bytes(cols));
            break;
        case PTQ_CALL_QUANTIZE_LAYER_PER_ROW:
            if (rows < 1) return 0;
            add((size_t)rows * sizeof(double));             // per-row losses
            break;
        case PTQ_CALL_QUANTIZE_LAYER_DYNAMIC:
            if (rows < 1) return 0;
            add(c * c * sizeof(double));                    // current matrix and the gathered one (ping-pong)
            add(c * c * sizeof(double));
            add((size_t)rows * c * sizeof(double));         // current weights and the gathered ones (ping-pong)
            add((size_t)rows * c * sizeof(double));
            add((size_t)rows * c * sizeof(double));         // scaled errors E
            add((size_t)rows * c * sizeof(double));         // dW
            add((size_t)rows * c);                          // codes of the block being swept
            add(c * sizeof(double));                        // scores
            add(c * sizeof(double));                        // diagonal
            add((size_t)cdiv(rows, kScoreRowChunk) * c * sizeof(double));
            add(c * sizeof(int32_t));                       // order of the round
            add(c * sizeof(int32_t));                       // original column of every position (ping-pong)
            add(c * sizeof(int32_t));
            add(loss_partials_count(rows, cols) * sizeof(double));
            add(2 * sizeof(unsigned));
            add(((size_t)cdiv(rows, kSweepRows) + 1) * sizeof(unsigned));
            add(chol_scratch_doubles(cols) * sizeof(double));
            break;
        default:
            return 0;
    }
    return total;
}

int ptq_hessian_accumulate_f64(double* H, const float* X, int cols, int n, int64_t ldx, void* ws, size_t ws_bytes,
                               int32_t* status, void* stream_) {
    (void)status;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!H || !X || cols < 1 || n < 1 || ldx < n) return PTQ_ERR_INVALID_ARG;
    if (cols > kMaxGridY) return PTQ_ERR_UNSUPPORTED;
    if (!aligned16(H) || !aligned16(ws)) return PTQ_ERR_ALIGNMENT;
    if (!ws || ws_bytes < ptq_workspace_bytes(PTQ_CALL_HESSIAN_ACCUMULATE_F64, 0, cols, n)) return PTQ_ERR_WORKSPACE;
    Carver cv(ws);
    double* Xd = cv.take<double>((size_t)cols * n);
    { Launch l(K_CONVERT_F64, stream); convert_f32_f64_kernel<<<dim3(grid_x_for(n, 256), cols), 256, 0, stream>>>(X, cols, n, ldx, Xd); }
    GemmParams g = gemm_defaults();
    g.A = Xd; g.lda = n; g.a_trans = 0;
    g.B = Xd; g.ldb = n; g.b_trans = 1;
    g.C = H; g.ldc = cols;
    g.M = cols; g.N = cols; g.K = n;
    g.alpha = 2.0; g.beta = 1.0; g.upper_only = 1; g.mirror = 1;
    return launch_dgemm(K_DGEMM_GRAM, g, 1, stream);
}

int ptq_hessian_accumulate(double* H, const float* X, int cols, int n, int64_t ldx, void* ws, size_t ws_bytes,
                           int32_t* status, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!H || !X || cols < 1 || n < 1 || ldx < n) return PTQ_ERR_INVALID_ARG;
    if (!aligned16(H) || !aligned16(ws)) return PTQ_ERR_ALIGNMENT;
    if (!ws || ws_bytes < ptq_workspace_bytes(PTQ_CALL_HESSIAN_ACCUMULATE, 0, cols, n)) return PTQ_ERR_WORKSPACE;
    GramSource src{};
    src.base = X; src.ldx = ldx;
    return gram_accumulate(H, src, cols, n, ws, status, stream);
}

int ptq_hessian_accumulate_conv(double* H, const float* act, int batch, int channels, int height, int width, int kh,
                                int kw, int stride, int pad, void* ws, size_t ws_bytes, int32_t* status,
                                void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!H || !act || batch < 1 || channels < 1 || height < 1 || width < 1 || kh < 1 || kw < 1 || stride < 1 || pad < 0)
        return PTQ_ERR_INVALID_ARG;
    if (height + 2 * pad < kh || width + 2 * pad < kw) return PTQ_ERR_INVALID_ARG;
    const int64_t oh = (height + 2 * pad - kh) / stride + 1, ow = (width + 2 * pad - kw) / stride + 1;
    const int64_t cols64 = (int64_t)channels * kh * kw, n64 = (int64_t)batch * oh * ow;
    if (cols64 > (1 << 20) || n64 > (int64_t)1 << 30) return PTQ_ERR_UNSUPPORTED;
    const int cols = (int)cols64, n = (int)n64;
    if (!aligned16(H) || !aligned16(ws)) return PTQ_ERR_ALIGNMENT;
    if (!ws || ws_bytes < ptq_workspace_bytes(PTQ_CALL_HESSIAN_ACCUMULATE, 0, cols, n)) return PTQ_ERR_WORKSPACE;
    GramSource src{};
    src.base = act; src.conv = 1;
    src.channels = channels; src.height = height; src.width = width;
    src.kh = kh; src.kw = kw; src.stride = stride; src.pad = pad; src.oh = (int)oh; src.ow = (int)ow;
    return gram_accumulate(H, src, cols, n, ws, status, stream);
}

int ptq_prepare_hinv(const double* H, int cols, int damp_mode, double damp, double* Hinv, double* Hinv_diag,
                     double* lambda_out, void* ws, size_t ws_bytes, int32_t* status, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!H || !Hinv || !Hinv_diag || !lambda_out || cols < 1 || !(damp >= 0.0)) return PTQ_ERR_INVALID_ARG;
    if (damp_mode != PTQ_DAMP_REL_MEAN_DIAG && damp_mode != PTQ_DAMP_ABS) return PTQ_ERR_INVALID_ARG;
    if (cols > kMaxGridY) return PTQ_ERR_UNSUPPORTED;                          // rows index the grid's y dimension
    if (!aligned16(H) || !aligned16(Hinv) || !aligned16(ws)) return PTQ_ERR_ALIGNMENT;
    if (!ws || ws_bytes < ptq_workspace_bytes(PTQ_CALL_PREPARE_HINV, 0, cols, 0)) return PTQ_ERR_WORKSPACE;
    const int n = cols;
    Carver cv(ws);
    double* R = cv.take<double>((size_t)n * n);
    double* V = cv.take<double>((size_t)n * n);
    unsigned* bar = cv.take<unsigned>(2);
    double* Dbuf = cv.take<double>(chol_scratch_doubles(n));
    void* pws = chol_panel_workspace_bytes(n) ? static_cast<void*>(cv.take<char>(chol_panel_workspace_bytes(n))) : nullptr;
    { Launch l(K_LAMBDA, stream); lambda_kernel<<<1, 256, 0, stream>>>(H, n, damp_mode, damp, lambda_out, status); }
    { Launch l(K_DAMP_COPY, stream); damp_copy_kernel<<<dim3(grid_x_for(n, 256), n), 256, 0, stream>>>(H, R, n, lambda_out); }
    // W = U^-T comes out of the factorisation sweep itself (V must start as zero)
    if (cudaMemsetAsync(V, 0, (size_t)n * n * sizeof(double), stream) != cudaSuccess) return PTQ_ERR_CUDA;
    int st = cholesky_upper_auto(R, n, V, Dbuf, bar, pws, status, stream);
    if (st) return st;
    if (n >= kSlicedMinCols && n <= kXMaxK && x_operand_bytes(n, n) <= (size_t)n * n * sizeof(double)) {
        // Hinv = W^T W on the int8 tensor path: the columns of the lower-triangular W are sliced once (into R, which is
        // free now) and serve as both operands; only k >= max(i, j) contributes, upper tiles computed and mirrored
        Carver rv(R);
        const XOperand w = x_slice_operand(rv, V, n, 1, n, n, stream);
        XGemmParams prm{};
        prm.C = Hinv; prm.ldc = n; prm.alpha = 1.0; prm.status = status;
        prm.out_mode = X_OUT_SYM; prm.k_mode = X_K_FROM_MAX;
        st = x_product(w, w, prm, stream);
    } else {
        st = lauum_lower(V, Hinv, n, stream);
    }
    if (st) return st;
    { Launch l(K_EXTRACT_DIAG, stream); extract_diag_kernel<<<cdiv(n, 256), 256, 0, stream>>>(Hinv, n, Hinv_diag); }
    return launch_status();
}

int ptq_minmax_grid(const float* W, int rows, int cols, int64_t ldw, int bits, float* scale, float* zero,
                    int32_t* status, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!W || !scale || !zero || rows < 1 || cols < 1 || ldw < cols || bits < 2 || bits > 8)
        return PTQ_ERR_INVALID_ARG;
    { Launch l(K_MINMAX_GRID, stream); minmax_grid_kernel<<<rows, 256, 0, stream>>>(W, rows, cols, ldw, bits, scale, zero, status); }
    return launch_status();
}

int ptq_sensitivity_order(const float* W, int rows, int cols, int64_t ldw, const double* Hinv_diag, const float* scale,
                          const float* zero, int bits, int score_mode, double* S, int32_t* perm, void* ws,
                          size_t ws_bytes, int32_t* status, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int bad = order_args_check(W, rows, cols, ldw, Hinv_diag, scale, zero, bits, score_mode, S, perm);
    if (bad) return bad;
    if (!ws || ws_bytes < ptq_workspace_bytes(PTQ_CALL_SENSITIVITY_ORDER, rows, cols, 0)) return PTQ_ERR_WORKSPACE;
    if (!aligned16(ws)) return PTQ_ERR_ALIGNMENT;
    Carver cv(ws);
    double* partial = cv.take<double>((size_t)cdiv(rows, kScoreRowChunk) * cols);
    return order_launch(W, rows, cols, ldw, Hinv_diag, scale, zero, bits, score_mode & ~PTQ_SCORE_ASCENDING,
                        (score_mode & PTQ_SCORE_ASCENDING) ? 1 : 0, S, perm, partial, status, stream);
}

int ptq_sensitivity_order_static(const float* W, int rows, int cols, int64_t ldw, const double* Hinv_diag,
                                 const float* scale, const float* zero, int bits, int score_mode, double* S,
                                 int32_t* perm, int32_t* status, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int bad = order_args_check(W, rows, cols, ldw, Hinv_diag, scale, zero, bits, score_mode, S, perm);
    if (bad) return bad;
    if ((size_t)cdiv(rows, kScoreRowChunk) * (size_t)cols > kStaticScratchDoubles) return PTQ_ERR_STATIC_SCRATCH;
    double* partial = nullptr;
    const int st = static_scratch_address(&partial);
    if (st) return st;
    // Every partial[ch][j] that score_final_kernel reads is written first by score_partial_kernel, so nothing
    // left in the array by an earlier call is ever used and nothing needs clearing.
    return order_launch(W, rows, cols, ldw, Hinv_diag, scale, zero, bits, score_mode & ~PTQ_SCORE_ASCENDING,
                        (score_mode & PTQ_SCORE_ASCENDING) ? 1 : 0, S, perm, partial, status, stream);
}

int ptq_quantize_layer_dynamic(const float* W, int rows, int cols, int64_t ldw, const double* Hinv, const float* scale,
                               const float* zero, int bits, int score_mode, int block, uint8_t* codes, float* What,
                               int32_t* order_out, const double* H_undamped, double* loss_out, void* ws,
                               size_t ws_bytes, int32_t* status, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!W || !Hinv || !scale || !zero || !codes || !order_out || rows < 1 || cols < 1 || ldw < cols || bits < 2 ||
        bits > 8 || block < 1)
        return PTQ_ERR_INVALID_ARG;
    if (score_mode & ~(PTQ_SCORE_ASCENDING | 7)) return PTQ_ERR_INVALID_ARG;
    const int mode = score_mode & ~PTQ_SCORE_ASCENDING, ascending = (score_mode & PTQ_SCORE_ASCENDING) ? 1 : 0;
    if (mode < PTQ_SCORE_QERR || mode > PTQ_SCORE_NONE) return PTQ_ERR_INVALID_ARG;
    if (block < cols && (block % kNB) != 0) return PTQ_ERR_UNSUPPORTED;     // rounds end on the 64-column block grid
    if (rows > kMaxGridY || cols > kMaxGridY || cdiv(rows, kScoreRowChunk) > kMaxGridY) return PTQ_ERR_UNSUPPORTED;
    if (!aligned16(Hinv) || !aligned16(ws)) return PTQ_ERR_ALIGNMENT;
    if (!ws || ws_bytes < ptq_workspace_bytes(PTQ_CALL_QUANTIZE_LAYER_DYNAMIC, rows, cols, 0)) return PTQ_ERR_WORKSPACE;
    const size_t c = (size_t)cols;
    Carver cv(ws);
    double* Abuf[2] = {cv.take<double>(c * c), nullptr};
    Abuf[1] = cv.take<double>(c * c);
    double* Wbuf[2] = {cv.take<double>((size_t)rows * c), nullptr};
    Wbuf[1] = cv.take<double>((size_t)rows * c);
    double* E = cv.take<double>((size_t)rows * c);
    double* dW = cv.take<double>((size_t)rows * c);
    uint8_t* codes_p = cv.take<uint8_t>((size_t)rows * c);
    double* S = cv.take<double>(c);
    double* diag = cv.take<double>(c);
    const int chunks = cdiv(rows, kScoreRowChunk);
    double* partial = cv.take<double>((size_t)chunks * c);
    int32_t* ordr = cv.take<int32_t>(c);
    int32_t* obuf[2] = {cv.take<int32_t>(c), nullptr};
    obuf[1] = cv.take<int32_t>(c);
    double* partials = cv.take<double>(loss_partials_count(rows, cols));
    unsigned* bar = cv.take<unsigned>(2);
    unsigned* sweep_flags = cv.take<unsigned>((size_t)cdiv(rows, kSweepRows) + 1);
    double* Dbuf = cv.take<double>(chol_scratch_doubles(cols));
    const bool want_loss = H_undamped && loss_out;

    { Launch l(K_DYN_AUX, stream); iota_kernel<<<cdiv(cols, 256), 256, 0, stream>>>(obuf[0], cols); }
    const int32_t* ocur = obuf[0];           // original column index of every current position
    // current state: the m columns still to do, their matrix (upper triangle valid) and their weights
    const double* Acur = Hinv;
    int64_t lda = cols;
    const double* Wcur = nullptr;            // round 0 reads the float32 weights
    int64_t ldc = 0;
    int m = cols, done = 0, cur = 0;
    while (m > 0) {
        const int b = block < m ? block : m;
        { Launch l(K_DYN_AUX, stream); extract_diag_ld_kernel<<<cdiv(m, 256), 256, 0, stream>>>(Acur, lda, m, diag); }
        if (mode != PTQ_SCORE_NONE) {
            Launch l(K_SCORE_PARTIAL, stream);
            if (Wcur)
                score_partial_kernel<double><<<dim3(cdiv(m, kScoreCols), chunks), 256, 0, stream>>>(Wcur, rows, m, ldc, scale,
                                                                                                zero, bits, mode, partial);
            else
                score_partial_kernel<float><<<dim3(cdiv(m, kScoreCols), chunks), 256, 0, stream>>>(W, rows, m, ldw, scale,
                                                                                               zero, bits, mode, partial);
        }
        { Launch l(K_SCORE_FINAL, stream); score_final_kernel<<<cdiv(m, 128), 128, 0, stream>>>(partial, chunks, m, diag, mode, S, status); }
        { Launch l(K_RANK_SORT, stream); rank_sort_kernel<<<cdiv(m, kRankCols), 256, 0, stream>>>(S, m, ascending, ordr, ocur); }
        double* An = Abuf[cur];
        double* Wn = Wbuf[cur];
        int32_t* onew = obuf[cur ^ 1];
        {
            Launch l(K_DYN_GATHER, stream);
            const int gy = m < 4096 ? m : 4096, gr = rows < 4096 ? rows : 4096;
            gather_upper_kernel<<<dim3(grid_x_for(m, 256), gy), 256, 0, stream>>>(Acur, lda, ordr, m, An);
            if (Wcur)
                gather_cols_kernel<double><<<dim3(grid_x_for(m, 256), gr), 256, 0, stream>>>(Wcur, ldc, rows, m, ordr, Wn);
            else
                gather_cols_kernel<float><<<dim3(grid_x_for(m, 256), gr), 256, 0, stream>>>(W, ldw, rows, m, ordr, Wn);
            gather_index_kernel<<<cdiv(m, 256), 256, 0, stream>>>(ocur, ordr, m, b, onew, order_out + done);
        }
        int st = cholesky_upper(An, m, nullptr, Dbuf, bar, status, stream, b < m ? b / kNB : 0);
        if (st) return st;
        st = sweep_launch(Wn, An, E, codes_p, scale, zero, rows, b, bits, sweep_flags, status, stream, m);
        if (st) return st;
        if (b < m) {
            // Eq. 11 for the columns still to come, all b columns at once: Wn[:, b:] -= E[:, :b] U[:b, b:]
            GemmParams g = gemm_defaults();
            g.A = E; g.lda = m; g.a_trans = 0;
            g.B = An + b; g.ldb = m; g.b_trans = 0;
            g.C = Wn + b; g.ldc = m;
            g.M = rows; g.N = m - b; g.K = b;
            g.alpha = -1.0; g.beta = 1.0;
            st = launch_dgemm(K_DGEMM_DYN, g, 1, stream);
            if (st) return st;
        }
        {
            Launch l(K_DYN_AUX, stream);
            const int gr = rows < 4096 ? rows : 4096;
            emit_block_kernel<<<dim3(grid_x_for(b, 256), gr), 256, 0, stream>>>(codes_p, m, onew, b, W, rows, cols, ldw,
                                                                            scale, zero, codes, What,
                                                                            want_loss ? dW : nullptr);
        }
        Acur = An + (size_t)b * m + b; lda = m;
        Wcur = Wn + b; ldc = m;
        // what is left of the gathered arrays is the next round's state; the next round gathers into the other buffers
        ocur = onew + b;
        done += b;
        m -= b;
        cur ^= 1;
    }
    if (want_loss) {
        GemmParams g = gemm_defaults();
        g.kend_mode = 1; g.sym_double = 1;
        g.A = dW; g.lda = cols; g.a_trans = 0;
        g.B = H_undamped; g.ldb = cols; g.b_trans = 0;
        g.M = rows; g.N = cols; g.K = cols;
        g.D = dW; g.ldd = cols; g.partials = partials;
        g.ksplit = loss_ksplit(rows, cols);
        dim3 grid;
        const int st = launch_dgemm(K_DGEMM_LOSS, g, 1, stream, 64, &grid);
        if (st) return st;
        { Launch l(K_SUM_PARTIALS, stream); sum_partials_kernel<<<1, 256, 0, stream>>>(partials, (int)(grid.x * grid.y * grid.z), 0.5, loss_out); }
    }
    return launch_status();
}

int ptq_quantize_layer_per_row(const float* W, int rows, int cols, int64_t ldw, const double* Hinv, const float* scale,
                               const float* zero, int bits, int score_mode, uint8_t* codes, float* What,
                               int32_t* perm_rows, const double* H_undamped, double* loss_out, void* ws,
                               size_t ws_bytes, int32_t* status, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!W || !Hinv || !scale || !zero || !codes || !perm_rows || rows < 1 || cols < 1 || ldw < cols || bits < 2 ||
        bits > 8)
        return PTQ_ERR_INVALID_ARG;
    if (score_mode & ~(PTQ_SCORE_ASCENDING | 7)) return PTQ_ERR_INVALID_ARG;
    const int mode = score_mode & ~PTQ_SCORE_ASCENDING, ascending = (score_mode & PTQ_SCORE_ASCENDING) ? 1 : 0;
    if (mode < PTQ_SCORE_QERR || mode > PTQ_SCORE_NONE) return PTQ_ERR_INVALID_ARG;
    if (cols > kPerRowMaxCols) return PTQ_ERR_UNSUPPORTED;       // one private inverse Hessian per CTA, in shared memory
    if (!ws || ws_bytes < ptq_workspace_bytes(PTQ_CALL_QUANTIZE_LAYER_PER_ROW, rows, cols, 0)) return PTQ_ERR_WORKSPACE;
    if (!aligned16(ws)) return PTQ_ERR_ALIGNMENT;
    DeviceState* dev = nullptr;
    int st = current_device_state(&dev);
    if (st) return st;
    st = ensure_smem_attr(dev, SA_SMALL, [] {
        return cudaFuncSetAttribute(per_row_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)per_row_smem_bytes(kPerRowMaxCols));
    });
    if (st) return st;
    Carver cv(ws);
    double* row_loss = cv.take<double>(rows);
    const bool want_loss = H_undamped && loss_out;
    {
        Launch l(K_PER_ROW, stream);
        per_row_kernel<<<rows, kPerRowThreads, per_row_smem_bytes(cols), stream>>>(
            W, rows, cols, ldw, Hinv, scale, zero, bits, mode, ascending, codes, What, perm_rows,
            want_loss ? H_undamped : nullptr, want_loss ? row_loss : nullptr, status);
    }
    if (want_loss) {
        Launch l(K_SUM_PARTIALS, stream);
        sum_partials_kernel<<<1, 256, 0, stream>>>(row_loss, rows, 1.0, loss_out);
    }
    return launch_status();
}

size_t ptq_gemm_nt_sliced_workspace_bytes(int m, int n, int k) {
    if (m < 1 || n < 1 || k < 1) return 0;
    return i8gemm_workspace_bytes(m, n, k);
}

int ptq_gemm_nt_sliced(double* C, int64_t ldc, const double* A, int64_t lda, const double* B, int64_t ldb, int b_is_kn,
                       int m, int n, int k, double alpha, void* ws, size_t ws_bytes, int32_t* status, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!C || !A || !B || m < 1 || n < 1 || k < 1 || ldc < n || lda < k || ldb < (b_is_kn ? n : k))
        return PTQ_ERR_INVALID_ARG;
    if (k > kXMaxK) return PTQ_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < i8gemm_workspace_bytes(m, n, k)) return PTQ_ERR_WORKSPACE;
    if (!aligned16(ws)) return PTQ_ERR_ALIGNMENT;
    return i8gemm_nt(C, ldc, A, lda, B, ldb, b_is_kn ? 1 : 0, m, n, k, alpha, ws, status, stream);
}

int ptq_sort_scores(const double* S, int cols, int ascending, int32_t* perm, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!S || !perm || cols < 1) return PTQ_ERR_INVALID_ARG;
    { Launch l(K_RANK_SORT, stream); rank_sort_kernel<<<cdiv(cols, kRankCols), 256, 0, stream>>>(S, cols, ascending ? 1 : 0, perm); }
    return launch_status();
}

int ptq_selftest_wait_timeout(int which, long long limit_cycles, void* ws, size_t ws_bytes, int32_t* status,
                              void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if ((which != 0 && which != 1) || limit_cycles < 1 || limit_cycles > kSpinLimitCycles || !status)
        return PTQ_ERR_INVALID_ARG;
    if (!ws || ws_bytes < 4 * sizeof(unsigned)) return PTQ_ERR_WORKSPACE;
    if (!aligned16(ws)) return PTQ_ERR_ALIGNMENT;
    unsigned* words = static_cast<unsigned*>(ws);
    if (cudaMemsetAsync(words, 0, 4 * sizeof(unsigned), stream) != cudaSuccess) return PTQ_ERR_CUDA;
    if (which == 1) {
        Launch l(K_SELFTEST, stream);
        selftest_counter_kernel<<<1, 32, 0, stream>>>(words, status, limit_cycles);
        return launch_status();
    }
    DeviceState* dev = nullptr;
    const int st = current_device_state(&dev);
    if (st) return st;
    if (!dev->coop) return PTQ_ERR_UNSUPPORTED;
    void* args[] = {&words, &status, &limit_cycles};
    Launch l(K_SELFTEST, stream);
    if (cudaLaunchCooperativeKernel((const void*)selftest_barrier_kernel, dim3(dev->sms), dim3(kCholThreads), args, 0,
                                    stream) != cudaSuccess) {
        cudaGetLastError();
        return PTQ_ERR_CUDA;
    }
    return PTQ_OK;
}

int ptq_fp64_probe(int kind, int iters, double* sink, double* flops_out, void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if ((kind != 0 && kind != 1) || iters < 1 || iters > (1 << 24) || !sink || !flops_out) return PTQ_ERR_INVALID_ARG;
    DeviceState* dev = nullptr;
    const int st = current_device_state(&dev);
    if (st) return st;
    const int grid = dev->sms * kProbeCtasPerSm;
    const double threads = (double)grid * kProbeThreads;
    Launch l(K_FP64_PROBE, stream);
    if (kind == 0) {
        fp64_probe_fma_kernel<<<grid, kProbeThreads, 0, stream>>>(iters, sink);
        *flops_out = threads * kProbeChains * (double)iters * 2.0;
    } else {
        fp64_probe_mma_kernel<<<grid, kProbeThreads, 0, stream>>>(iters, sink);
        *flops_out = (threads / 32.0) * kProbeChains * (double)iters * (8.0 * 8.0 * 4.0 * 2.0);
    }
    return launch_status();
}

int ptq_quantize_layer(const float* W, int rows, int cols, int64_t ldw, const double* Hinv, const int32_t* perm,
                       const float* scale, const float* zero, int bits, uint8_t* codes, float* What,
                       const double* H_undamped, double* loss_out, void* ws, size_t ws_bytes, int32_t* status,
                       void* stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (!W || !Hinv || !perm || !scale || !zero || !codes || rows < 1 || cols < 1 || ldw < cols || bits < 2 ||
        bits > 8)
        return PTQ_ERR_INVALID_ARG;
    if (rows > kMaxGridY || cols > kMaxGridY) return PTQ_ERR_UNSUPPORTED;     // rows / columns index the grid's y dimension
    if (!aligned16(Hinv) || !aligned16(ws)) return PTQ_ERR_ALIGNMENT;
    if (!ws || ws_bytes < ptq_workspace_bytes(PTQ_CALL_QUANTIZE_LAYER, rows, cols, 0)) return PTQ_ERR_WORKSPACE;
    const int n = cols;
    Carver cv(ws);
    double* U = cv.take<double>((size_t)n * n);
    double* Wp = cv.take<double>((size_t)rows * n);
    double* E = cv.take<double>((size_t)rows * n);
    uint8_t* codes_p = cv.take<uint8_t>((size_t)rows * n);
    int32_t* flags = cv.take<int32_t>(n);
    int32_t* invperm = cv.take<int32_t>(n);
    double* partials = cv.take<double>(loss_partials_count(rows, cols));
    unsigned* bar = cv.take<unsigned>(2);
    unsigned* sweep_flags = cv.take<unsigned>((size_t)cdiv(rows, kSweepRows) + 1);
    double* Dbuf = cv.take<double>(chol_scratch_doubles(n));
    void* xws = (rows >= kSuperBlockMinRows && n >= 4 * kSuperBlock)
                    ? static_cast<void*>(cv.take<char>(i8gemm_workspace_bytes(rows, n, kSuperBlock))) : nullptr;
    void* pws = chol_panel_workspace_bytes(n) ? static_cast<void*>(cv.take<char>(chol_panel_workspace_bytes(n))) : nullptr;

    // flags and invperm are adjacent pieces of the workspace: clear both
    if (cudaMemsetAsync(flags, 0, (size_t)((char*)invperm - (char*)flags) + (size_t)n * sizeof(int32_t), stream) !=
        cudaSuccess)
        return PTQ_ERR_CUDA;
    { Launch l(K_PERM_CHECK, stream); perm_check_kernel<<<cdiv(n, 256), 256, 0, stream>>>(perm, n, flags, invperm, status); }
    { Launch l(K_GATHER_SYM, stream); gather_sym_kernel<<<dim3(grid_x_for(n, 256), n), 256, 0, stream>>>(Hinv, perm, n, U); }
    { Launch l(K_GATHER_W, stream); gather_w_kernel<<<dim3(grid_x_for(n, 256), rows), 256, 0, stream>>>(W, rows, n, ldw, perm, Wp); }
    int st = cholesky_upper_auto(U, n, nullptr, Dbuf, bar, pws, status, stream);   // blocked Eq. 12
    if (st) return st;

    if (rows >= kSuperBlockMinRows && n >= 4 * kSuperBlock) {
        // Tall and wide layers: the deferred part of Eq. 11 dominates (rows cols^2 / 2 multiply-adds), and inside the sweep
        // kernel it runs as 32 x 64 x 64 tiles.  The columns are therefore swept in super-blocks of 1024; what a
        // super-block owes to all later columns is applied by one large product, W[:, later] -= E[:, sb] U[sb, later],
        // with k = 1024.
        for (int off = 0; off < n; off += kSuperBlock) {
            const int sb = n - off < kSuperBlock ? n - off : kSuperBlock;
            st = sweep_launch(Wp + off, U + (size_t)off * n + off, E + off, codes_p + off, scale, zero, rows, sb, bits,
                              sweep_flags, status, stream, n);
            if (st) return st;
            if (off + sb < n) {
                // W[:, later] -= E[:, sb] U[sb, later] on the int8 tensor path (i8gemm.cuh), float64-accurate
                st = i8gemm_nt(Wp + off + sb, n, E + off, n, U + (size_t)off * n + off + sb, n, 1, rows, n - off - sb, sb,
                               -1.0, xws, status, stream);
                if (st) return st;
            }
        }
    } else {
        st = sweep_launch(Wp, U, E, codes_p, scale, zero, rows, n, bits, sweep_flags, status, stream);
        if (st) return st;
    }

    const bool want_loss = H_undamped && loss_out;
    double* dW = want_loss ? Wp : nullptr;
    {
        Launch l(K_FINALIZE, stream);
        finalize_kernel<<<dim3(grid_x_for(n, 256), rows), 256, 0, stream>>>(codes_p, invperm, W, rows, n, ldw, scale,
                                                                           zero, codes, What, dW);
    }
    if (want_loss && rows >= kSuperBlockMinRows && n >= kSlicedMinCols && n <= kXMaxK &&
        x_operand_bytes(rows, n) <= (size_t)rows * n * sizeof(double) &&
        x_operand_bytes(n, n) <= (size_t)n * n * sizeof(double) &&
        2 * (size_t)x_num_tiles(rows, n) <= loss_partials_count(rows, cols)) {
        // 1/2 sum_ij dW_ij (dW H)_ij on the int8 tensor path.  H is symmetric: per 64-column block j the column blocks
        // k < j count twice (they stand in for the blocks k > j as well) and the block k = j once, so two products
        // with reduction epilogues, k before the tile's own block (weight 2 * 1/2) and k in it (weight 1/2).
        // The slices of dW go where E was, those of H where U was: both are free now.
        Carver ev(E), uv(U);
        const XOperand a = x_slice_operand(ev, dW, n, 0, rows, n, stream);
        const XOperand b = x_slice_operand(uv, H_undamped, n, 0, n, n, stream);
        const int tiles = x_num_tiles(rows, n);
        XGemmParams prm{};
        prm.status = status; prm.out_mode = X_OUT_REDUCE; prm.D = dW; prm.ldd = n;
        prm.k_mode = X_K_BEFORE_J; prm.alpha = 1.0; prm.partials = partials;
        st = x_product(a, b, prm, stream);
        if (st) return st;
        prm.k_mode = X_K_OWN_J; prm.alpha = 0.5; prm.partials = partials + tiles;
        st = x_product(a, b, prm, stream);
        if (st) return st;
        { Launch l(K_SUM_PARTIALS, stream); sum_partials_kernel<<<1, 256, 0, stream>>>(partials, 2 * tiles, 1.0, loss_out); }
    } else if (want_loss) {
        // sum_ic dW_ic (dW H)_ic; H is symmetric, so for the 64-column block of c only k up to the end of that block is
        // summed and the blocks before it are doubled
        GemmParams g = gemm_defaults();
        g.kend_mode = 1; g.sym_double = 1;
        g.A = dW; g.lda = n; g.a_trans = 0;
        g.B = H_undamped; g.ldb = n; g.b_trans = 0;
        g.M = rows; g.N = n; g.K = n;
        g.D = dW; g.ldd = n; g.partials = partials;
        g.ksplit = loss_ksplit(rows, n);
        dim3 grid;
        st = launch_dgemm(K_DGEMM_LOSS, g, 1, stream, 64, &grid);
        if (st) return st;
        { Launch l(K_SUM_PARTIALS, stream); sum_partials_kernel<<<1, 256, 0, stream>>>(partials, (int)(grid.x * grid.y * grid.z), 0.5, loss_out); }
    }
    return launch_status();
}

}  // extern "C"
