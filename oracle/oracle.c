/*
 * Float64 CPU oracle for the sensitivity-ordered, row-parallel layer quantizer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * method computes, written from the paper's text.  It shares no code, header,
 * table or helper with the CUDA library; only tests, the smoke check and the
 * bench's CPU-baseline leg may call it.
 *
 * Conventions
 *   W   [rows x cols]  float32, row-major, leading dimension ldw   (Sec. 3: d_row x d_col)
 *   X   [cols x n]     float32, row-major, leading dimension ldx   (Sec. 3: d_col x N)
 *   H, Hinv [cols x cols] float64, row-major, full symmetric storage
 * All arithmetic is IEEE float64 (float32 inputs are converted exactly); every sum runs
 * over its index in ascending order.  OpenMP, when enabled, only distributes independent
 * rows / columns over threads and never changes the order of any sum.
 *
 * Pins (tests/test_oracle_pins.py): identity Hessian => round-to-nearest; every Eq. 12
 * update equals direct inversion of the remaining sub-matrix; Eq. 11 equals the constrained
 * least-squares minimiser; damped-loss sum identity; brute-force enumeration on tiny rows;
 * hand-worked ordering example; Gram / inverse against library routines; the factor-form mode
 * against the literal loop and a library Cholesky; dynamic re-ranking against its definition
 * replayed through the literal loop; the per-row mode against the hand example and single-row runs.
 * Parity unpinned: the greedy rounding decisions of a general layer have no external
 * definition beyond "nearest level of the compensated value"; they are pinned only through
 * the quantities that determine them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_OK = 0, ORACLE_ERR_INVALID_ARG = 1, ORACLE_ERR_NOT_SPD = 4, ORACLE_ERR_NOMEM = 9 };
enum { DAMP_REL_MEAN_DIAG = 0, DAMP_ABS = 1 };
enum { SCORE_QERR = 0, SCORE_PRUNE = 1, SCORE_ERR = 2, SCORE_W = 3, SCORE_NONE = 4, SCORE_ASCENDING = 16 };

int oracle_version(void) { return 1; }

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------------------------------
 * Sec. 3: for a convolutional layer d_col is the number of weights of one filter, so the
 * columns of X are the input patches those weights see.  Writes them out by definition:
 *   X[(c*kh + ki)*kw + kj][(b*oh + oy)*ow + ox] = act[b][c][oy*stride + ki - pad][ox*stride + kj - pad]
 * (zero outside the image), act = [batch][channels][height][width], X = [channels*kh*kw][batch*oh*ow],
 * oh = (height + 2 pad - kh)/stride + 1, ow alike.  No arithmetic: the Hessian of a convolution
 * is oracle_hessian_accumulate of this matrix.
 * ------------------------------------------------------------------------------------- */
int oracle_unfold(float *X, const float *act, int batch, int channels, int height, int width, int kh, int kw,
                  int stride, int pad) {
    if (!X || !act || batch < 1 || channels < 1 || height < 1 || width < 1 || kh < 1 || kw < 1 || stride < 1 ||
        pad < 0 || height + 2 * pad < kh || width + 2 * pad < kw)
        return ORACLE_ERR_INVALID_ARG;
    const int oh = (height + 2 * pad - kh) / stride + 1, ow = (width + 2 * pad - kw) / stride + 1;
    const size_t n = (size_t)batch * oh * ow;
    for (int c = 0; c < channels; ++c)
        for (int ki = 0; ki < kh; ++ki)
            for (int kj = 0; kj < kw; ++kj) {
                float *row = X + ((size_t)(c * kh + ki) * kw + kj) * n;
                for (int b = 0; b < batch; ++b)
                    for (int oy = 0; oy < oh; ++oy)
                        for (int ox = 0; ox < ow; ++ox) {
                            const int iy = oy * stride + ki - pad, ix = ox * stride + kj - pad;
                            float v = 0.0f;
                            if (iy >= 0 && iy < height && ix >= 0 && ix < width)
                                v = act[(((size_t)b * channels + c) * height + iy) * width + ix];
                            row[((size_t)b * oh + oy) * ow + ox] = v;
                        }
            }
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Sec. 3, Eq. 2: the layer error is ||W X - What X||^2, so its second derivative with
 * respect to one row of W is H = 2 X X^T.  Accumulates H += 2 * X X^T.
 * Each H[i][j] is the serial sum over n = 0..n-1 of X[i][n] * X[j][n].
 * ------------------------------------------------------------------------------------- */
int oracle_hessian_accumulate(double *H, const float *X, int cols, int n, int64_t ldx) {
    if (!H || !X || cols < 1 || n < 1 || ldx < n) return ORACLE_ERR_INVALID_ARG;
    /* Xt[k][j] = (double) X[j][k]: a transposed float64 copy so that the loop over j is contiguous. */
    double *Xt = (double *)malloc((size_t)n * cols * sizeof(double));
    if (!Xt) return ORACLE_ERR_NOMEM;
    for (int j = 0; j < cols; ++j)
        for (int k = 0; k < n; ++k) Xt[(size_t)k * cols + j] = (double)X[(size_t)j * ldx + k];
    int fail = 0;
#pragma omp parallel
    {
        double *acc = (double *)malloc((size_t)cols * sizeof(double));
        if (!acc) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(dynamic, 4)
            for (int i = 0; i < cols; ++i) {
                for (int j = i; j < cols; ++j) acc[j] = 0.0;
                for (int k = 0; k < n; ++k) { /* ascending n for every (i, j) */
                    const double xi = Xt[(size_t)k * cols + i];
                    const double *xr = Xt + (size_t)k * cols;
                    for (int j = i; j < cols; ++j) acc[j] += xi * xr[j];
                }
                for (int j = i; j < cols; ++j) {
                    const double add = 2.0 * acc[j];
                    H[(size_t)i * cols + j] += add;
                    if (j != i) H[(size_t)j * cols + i] += add; /* same products, same order */
                }
            }
        }
        free(acc);
    }
    free(Xt);
    return fail ? ORACLE_ERR_NOMEM : ORACLE_OK;
}

/* One entry of 2 X X^T, for sampled checks at sizes where the full matrix is too slow. */
double oracle_hessian_entry(const float *X, int n, int64_t ldx, int i, int j) {
    double s = 0.0;
    for (int k = 0; k < n; ++k) s += (double)X[(size_t)i * ldx + k] * (double)X[(size_t)j * ldx + k];
    return 2.0 * s;
}

/* ---------------------------------------------------------------------------------------
 * Implementation details (damping added to the diagonal) and Sec. 5 item 1 (Cholesky
 * decomposition, then the inverse of the factor).
 *   lambda = damp * mean_j H[j][j]   (relative mode)   or   lambda = damp   (absolute mode)
 *   Hd = H + lambda I = L L^T,  Y = L^{-1} by forward substitution,  Hinv = Y^T Y.
 * info[0] receives the failing pivot index when the matrix is not positive definite.
 * ------------------------------------------------------------------------------------- */
int oracle_prepare_hinv(const double *H, int cols, int mode, double damp, double *Hinv,
                        double *Hinv_diag, double *lambda_out, int *info) {
    if (!H || !Hinv || cols < 1 || !(damp >= 0.0)) return ORACLE_ERR_INVALID_ARG;
    const size_t n = (size_t)cols;
    double lambda;
    if (mode == DAMP_REL_MEAN_DIAG) {
        double tr = 0.0;
        for (size_t j = 0; j < n; ++j) tr += H[j * n + j];
        lambda = damp * (tr / (double)cols);
    } else if (mode == DAMP_ABS) {
        lambda = damp;
    } else {
        return ORACLE_ERR_INVALID_ARG;
    }
    if (lambda_out) *lambda_out = lambda;

    double *L = (double *)calloc(n * n, sizeof(double));
    double *Yt = (double *)calloc(n * n, sizeof(double)); /* Yt[c][k] = Y[k][c] */
    if (!L || !Yt) { free(L); free(Yt); return ORACLE_ERR_NOMEM; }

    /* Cholesky, column by column. */
    int bad = -1;
    for (size_t j = 0; j < n && bad < 0; ++j) {
        double s = H[j * n + j] + lambda;
        for (size_t k = 0; k < j; ++k) s -= L[j * n + k] * L[j * n + k];
        if (!(s > 0.0) || !isfinite(s)) { bad = (int)j; break; }
        const double ljj = sqrt(s);
        L[j * n + j] = ljj;
#pragma omp parallel for schedule(static)
        for (size_t i = j + 1; i < n; ++i) {
            double t = H[i * n + j];
            for (size_t k = 0; k < j; ++k) t -= L[i * n + k] * L[j * n + k];
            L[i * n + j] = t / ljj;
        }
    }
    if (bad >= 0) {
        if (info) info[0] = bad;
        free(L); free(Yt);
        return ORACLE_ERR_NOT_SPD;
    }

    /* Forward substitution L Y = I, one column c of Y at a time. */
#pragma omp parallel for schedule(dynamic, 8)
    for (size_t c = 0; c < n; ++c) {
        double *y = Yt + c * n;
        y[c] = 1.0 / L[c * n + c];
        for (size_t i = c + 1; i < n; ++i) {
            double t = 0.0;
            for (size_t k = c; k < i; ++k) t += L[i * n + k] * y[k];
            y[i] = -t / L[i * n + i];
        }
    }

    /* Hinv = Y^T Y; Y is lower triangular so the sum starts at max(a, b). */
#pragma omp parallel for schedule(dynamic, 8)
    for (size_t a = 0; a < n; ++a) {
        for (size_t b = a; b < n; ++b) {
            double t = 0.0;
            for (size_t k = b; k < n; ++k) t += Yt[a * n + k] * Yt[b * n + k];
            Hinv[a * n + b] = t;
            Hinv[b * n + a] = t;
        }
    }
    if (Hinv_diag)
        for (size_t j = 0; j < n; ++j) Hinv_diag[j] = Hinv[j * n + j];
    free(L); free(Yt);
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * The grid (OBQ paragraph of Sec. 3: a fixed grid of width Delta, weights rounded onto it).
 * Reading taken: per-row asymmetric min-max range that always contains 0, computed once from
 * the original weights; the float32 scale / zero-point are what both sides then consume.
 * ------------------------------------------------------------------------------------- */
int oracle_minmax_grid(const float *W, int rows, int cols, int64_t ldw, int bits, float *scale,
                       float *zero) {
    if (!W || !scale || !zero || rows < 1 || cols < 1 || ldw < cols || bits < 2 || bits > 8)
        return ORACLE_ERR_INVALID_ARG;
    const double levels = (double)((1 << bits) - 1);
    for (int i = 0; i < rows; ++i) {
        double lo = 0.0, hi = 0.0;
        for (int j = 0; j < cols; ++j) {
            const double w = (double)W[(size_t)i * ldw + j];
            if (w < lo) lo = w;
            if (w > hi) hi = w;
        }
        if (hi == lo) { scale[i] = 1.0f; zero[i] = 0.0f; continue; }
        const double s = (hi - lo) / levels;
        scale[i] = (float)s;
        zero[i] = (float)rint(-lo / s);
    }
    return ORACLE_OK;
}

/* quant(w): nearest grid level (ties to even), clamped to the code range. */
static inline int quant_code(double w, double scale, double zero, int maxq) {
    double c = rint(w / scale) + zero;
    if (c < 0.0) c = 0.0;
    if (c > (double)maxq) c = (double)maxq;
    return (int)c;
}
static inline double dequant(int c, double scale, double zero) { return scale * ((double)c - zero); }

/* Exposed for the brute-force pins. */
int oracle_quant_code(double w, float scale, float zero, int bits) {
    return quant_code(w, (double)scale, (double)zero, (1 << bits) - 1);
}

/* ---------------------------------------------------------------------------------------
 * Sec. 4.2 steps 1-3.  Per-weight sensitivity (Eq. 10 for quantization, Eq. 8 for the
 * pruning form) from the ORIGINAL weights and the diagonal of the initial inverse Hessian;
 * column score S_j = sum over rows; columns sorted by S descending, equal scores keep the
 * lower column index first.
 *   QERR : (w - quant(w))^2 / (2 [Hinv]_jj)       PRUNE : w^2 / (2 [Hinv]_jj)
 *   ERR  : (w - quant(w))^2                        W     : w^2
 *   NONE : S_j = 0, identity order
 * Sec. 4.1 names every key in a descending ("des") and an ascending ("asc") variant: with
 * SCORE_ASCENDING added to the mode the columns are sorted by S ascending instead (equal scores
 * still keep the lower column index first).
 * ------------------------------------------------------------------------------------- */
static const double *g_sort_keys;
static int g_sort_ascending;
static int cmp_score_stable(const void *pa, const void *pb) {
    const int a = *(const int *)pa, b = *(const int *)pb;
    const double ka = g_sort_keys[a], kb = g_sort_keys[b];
    if (ka != kb) {
        const int a_first = g_sort_ascending ? (ka < kb) : (ka > kb);
        return a_first ? -1 : 1;
    }
    return (a > b) - (a < b);
}

int oracle_sensitivity_order(const float *W, int rows, int cols, int64_t ldw, const double *Hinv_diag,
                             const float *scale, const float *zero, int bits, int mode_and_direction,
                             double *S, int32_t *perm) {
    if (!W || !S || !perm || rows < 1 || cols < 1 || ldw < cols || bits < 2 || bits > 8)
        return ORACLE_ERR_INVALID_ARG;
    const int ascending = (mode_and_direction & SCORE_ASCENDING) != 0;
    const int mode = mode_and_direction & ~SCORE_ASCENDING;
    if (mode < 0 || mode > SCORE_NONE) return ORACLE_ERR_INVALID_ARG;
    if ((mode == SCORE_QERR || mode == SCORE_PRUNE) && !Hinv_diag) return ORACLE_ERR_INVALID_ARG;
    if ((mode == SCORE_QERR || mode == SCORE_ERR) && (!scale || !zero)) return ORACLE_ERR_INVALID_ARG;
    const int maxq = (1 << bits) - 1;
#pragma omp parallel for schedule(static)
    for (int j = 0; j < cols; ++j) {
        double s = 0.0;
        if (mode != SCORE_NONE) {
            for (int i = 0; i < rows; ++i) { /* ascending row index */
                const double w = (double)W[(size_t)i * ldw + j];
                double num;
                if (mode == SCORE_QERR || mode == SCORE_ERR) {
                    const double sc = (double)scale[i], zp = (double)zero[i];
                    const double q = dequant(quant_code(w, sc, zp, maxq), sc, zp);
                    num = (w - q) * (w - q);
                } else {
                    num = w * w;
                }
                if (mode == SCORE_QERR || mode == SCORE_PRUNE) s += num / (2.0 * Hinv_diag[j]);
                else s += num;
            }
        }
        S[j] = s;
    }
    for (int j = 0; j < cols; ++j) {
        if (!isfinite(S[j])) return ORACLE_ERR_INVALID_ARG;
        perm[j] = j;
    }
    g_sort_keys = S;
    g_sort_ascending = ascending;
    qsort(perm, (size_t)cols, sizeof(int32_t), cmp_score_stable);
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Sec. 4.2 steps 3-5 with Eq. 11 and Eq. 12 applied literally, one column at a time.
 *
 *   Wp = W[:, perm],  A = Hinv[perm][:, perm]
 *   for p = 0 .. cols-1:
 *       d = A[p][p]
 *       every row i:  c = quant code of Wp[i][p],  q = its grid value,  e_i = (Wp[i][p] - q) / d
 *       every row i, every j > p:  Wp[i][j] -= e_i * A[p][j]                     (Eq. 11)
 *       Wp[i][p] = q
 *       every j, k > p:  A[j][k] -= (A[j][p] / d) * A[p][k]                      (Eq. 12)
 *       row and column p of A become zero (that is what Eq. 12 leaves there)
 *   codes / What go back to the original column order; What is rounded to float32.
 *
 * Optional arguments (NULL to skip):
 *   H_undamped + loss_out : loss = 1/2 tr(dW H dW^T) with dW = W - What(float32)
 *   forced_codes [rows x cols, original column order]: use these codes instead of rounding
 *                 (the compensation still follows Eq. 11 / Eq. 12)
 *   prer  [rows x cols, original order]: the value Wp[i][p] / scale_i seen just before rounding
 *   A_trace [cols x cols x cols]: copy of A after the update of step p (tiny layers only)
 *   W_trace [cols x rows x cols]: copy of Wp after step p (permuted order)
 *   damped_sum_out: sum_i sum_p (Wp[i][p] - q)^2 / (2 d)  (the accumulated Eq. 10 increases)
 * ------------------------------------------------------------------------------------- */
int oracle_quantize_layer_ex(const float *W, int rows, int cols, int64_t ldw, const double *Hinv,
                             const int32_t *perm, const float *scale, const float *zero, int bits,
                             uint8_t *codes, float *What, const double *H_undamped, double *loss_out,
                             const uint8_t *forced_codes, double *prer, double *A_trace,
                             double *W_trace, double *damped_sum_out) {
    if (!W || !Hinv || !perm || !scale || !zero || !codes || rows < 1 || cols < 1 || ldw < cols ||
        bits < 2 || bits > 8)
        return ORACLE_ERR_INVALID_ARG;
    const size_t n = (size_t)cols, m = (size_t)rows;
    const int maxq = (1 << bits) - 1;
    {   /* perm must be a permutation */
        uint8_t *seen = (uint8_t *)calloc(n, 1);
        if (!seen) return ORACLE_ERR_NOMEM;
        int ok = 1;
        for (size_t j = 0; j < n; ++j) {
            if (perm[j] < 0 || perm[j] >= cols || seen[perm[j]]) { ok = 0; break; }
            seen[perm[j]] = 1;
        }
        free(seen);
        if (!ok) return ORACLE_ERR_INVALID_ARG;
    }
    double *A = (double *)malloc(n * n * sizeof(double));
    double *Wp = (double *)malloc(m * n * sizeof(double));
    double *e = (double *)malloc(m * sizeof(double));
    double *tcol = (double *)malloc(n * sizeof(double));
    double *dsum = (double *)calloc(m, sizeof(double));
    uint8_t *Cp = (uint8_t *)malloc(m * n);
    if (!A || !Wp || !e || !tcol || !dsum || !Cp) {
        free(A); free(Wp); free(e); free(tcol); free(dsum); free(Cp);
        return ORACLE_ERR_NOMEM;
    }
    for (size_t a = 0; a < n; ++a)
        for (size_t b = 0; b < n; ++b) A[a * n + b] = Hinv[(size_t)perm[a] * n + (size_t)perm[b]];
    for (size_t i = 0; i < m; ++i)
        for (size_t j = 0; j < n; ++j) Wp[i * n + j] = (double)W[i * (size_t)ldw + (size_t)perm[j]];

    int status = ORACLE_OK;
    for (size_t p = 0; p < n; ++p) {
        const double d = A[p * n + p];
        if (!(d > 0.0) || !isfinite(d)) { status = ORACLE_ERR_NOT_SPD; break; }
        const double *Ap = A + p * n;
#pragma omp parallel for schedule(static)
        for (size_t i = 0; i < m; ++i) {
            double *w = Wp + i * n;
            const double sc = (double)scale[i], zp = (double)zero[i];
            if (prer) prer[i * n + (size_t)perm[p]] = w[p] / sc;
            const int c = forced_codes ? (int)forced_codes[i * n + (size_t)perm[p]]
                                       : quant_code(w[p], sc, zp, maxq);
            const double q = dequant(c, sc, zp);
            const double diff = w[p] - q;
            dsum[i] += diff * diff / (2.0 * d);
            const double ei = diff / d;
            e[i] = ei;
            for (size_t j = p + 1; j < n; ++j) w[j] -= ei * Ap[j]; /* Eq. 11 */
            w[p] = q;
            Cp[i * n + p] = (uint8_t)c;
        }
        for (size_t j = p + 1; j < n; ++j) tcol[j] = A[j * n + p] / d;
#pragma omp parallel for schedule(static)
        for (size_t j = p + 1; j < n; ++j) { /* Eq. 12 */
            double *Aj = A + j * n;
            const double t = tcol[j];
            for (size_t k = p + 1; k < n; ++k) Aj[k] -= t * Ap[k];
        }
        for (size_t j = 0; j < n; ++j) { A[p * n + j] = 0.0; A[j * n + p] = 0.0; }
        if (A_trace) memcpy(A_trace + p * n * n, A, n * n * sizeof(double));
        if (W_trace) memcpy(W_trace + p * m * n, Wp, m * n * sizeof(double));
    }

    if (status == ORACLE_OK) {
        for (size_t i = 0; i < m; ++i)
            for (size_t p = 0; p < n; ++p) {
                const size_t j = (size_t)perm[p];
                codes[i * n + j] = Cp[i * n + p];
                if (What) What[i * n + j] = (float)Wp[i * n + p];
            }
        if (damped_sum_out) {
            double s = 0.0;
            for (size_t i = 0; i < m; ++i) s += dsum[i];
            *damped_sum_out = s;
        }
        if (H_undamped && loss_out) {
            /* 1/2 * sum_i dW_i H dW_i^T with dW measured against the float32 result */
            double *rowloss = (double *)calloc(m, sizeof(double));
            if (!rowloss) status = ORACLE_ERR_NOMEM;
            else {
#pragma omp parallel for schedule(static)
                for (size_t i = 0; i < m; ++i) {
                    double *dw = (double *)malloc(n * sizeof(double));
                    if (!dw) continue;
                    for (size_t p = 0; p < n; ++p) {
                        const size_t j = (size_t)perm[p];
                        dw[j] = (double)W[i * (size_t)ldw + j] - (double)(float)Wp[i * n + p];
                    }
                    double acc = 0.0;
                    for (size_t a = 0; a < n; ++a) {
                        double t = 0.0;
                        for (size_t b = 0; b < n; ++b) t += H_undamped[a * n + b] * dw[b];
                        acc += dw[a] * t;
                    }
                    rowloss[i] = 0.5 * acc;
                    free(dw);
                }
                double s = 0.0;
                for (size_t i = 0; i < m; ++i) s += rowloss[i];
                *loss_out = s;
                free(rowloss);
            }
        }
    }
    free(A); free(Wp); free(e); free(tcol); free(dsum); free(Cp);
    return status;
}

/* Eq. 2 evaluated directly from the calibration inputs: sum_i sum_n ((W - What) X)[i][n]^2. */
double oracle_loss_direct(const float *W, const float *What, int rows, int cols, int64_t ldw,
                          int64_t ldwh, const float *X, int n, int64_t ldx) {
    double *rowsum = (double *)calloc((size_t)rows, sizeof(double));
    if (!rowsum) return NAN;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < rows; ++i) {
        double s = 0.0;
        for (int k = 0; k < n; ++k) {
            double y = 0.0;
            for (int j = 0; j < cols; ++j)
                y += ((double)W[(size_t)i * ldw + j] - (double)What[(size_t)i * ldwh + j]) *
                     (double)X[(size_t)j * ldx + k];
            s += y * y;
        }
        rowsum[i] = s;
    }
    double total = 0.0;
    for (int i = 0; i < rows; ++i) total += rowsum[i];
    free(rowsum);
    return total;
}

/* ---------------------------------------------------------------------------------------
 * Factor form of the column loop, for layers too wide for the literal Eq. 12 loop (which costs
 * cols^3 / 3 multiply-adds over a cols^2 matrix whatever the number of rows).
 *
 * Eq. 12 is one step of a right-looking Cholesky factorisation: with A = Hinv[perm][:, perm] = U^T U
 * (U upper triangular), the matrix that Eq. 12 leaves before step p has row p equal to
 * U[p][p] * U[p][p:], so Eq. 11 for column p reads
 *     e_i = (w_ip - q_ip) / U[p][p],    w_ij -= e_i * U[p][j]   (j > p).
 * This mode is licensed only by its pins: tests/test_oracle_pins.py shows it equal to the literal
 * loop of oracle_quantize_layer_ex (codes, What, pre-rounding values) on every size the literal
 * loop reaches; the literal loop stays the definition.
 *
 * oracle_factor_upper: A = L L^T column by column (the same plain Cholesky as in oracle_prepare_hinv,
 * every sum in ascending index order), U[p][j] = L[j][p]; the strictly lower part of U is zero.
 * ------------------------------------------------------------------------------------- */
int oracle_factor_upper(const double *Hinv, const int32_t *perm, int cols, double *U, int *info) {
    if (!Hinv || !perm || !U || cols < 1) return ORACLE_ERR_INVALID_ARG;
    const size_t n = (size_t)cols;
    for (size_t j = 0; j < n; ++j)
        if (perm[j] < 0 || perm[j] >= cols) return ORACLE_ERR_INVALID_ARG;
    double *L = (double *)calloc(n * n, sizeof(double));
    if (!L) return ORACLE_ERR_NOMEM;
    int bad = -1;
    for (size_t j = 0; j < n && bad < 0; ++j) {
        double s = Hinv[(size_t)perm[j] * n + (size_t)perm[j]];
        for (size_t k = 0; k < j; ++k) s -= L[j * n + k] * L[j * n + k];
        if (!(s > 0.0) || !isfinite(s)) { bad = (int)j; break; }
        const double ljj = sqrt(s);
        L[j * n + j] = ljj;
#pragma omp parallel for schedule(static)
        for (size_t i = j + 1; i < n; ++i) {
            double t = Hinv[(size_t)perm[i] * n + (size_t)perm[j]];
            for (size_t k = 0; k < j; ++k) t -= L[i * n + k] * L[j * n + k];
            L[i * n + j] = t / ljj;
        }
    }
    if (bad >= 0) {
        if (info) info[0] = bad;
        free(L);
        return ORACLE_ERR_NOT_SPD;
    }
    for (size_t p = 0; p < n; ++p)
        for (size_t j = 0; j < n; ++j) U[p * n + j] = j >= p ? L[j * n + p] : 0.0;
    free(L);
    return ORACLE_OK;
}

/* The sweep of Sec. 4.2 steps 4-5 on the given rows with the factor U of oracle_factor_upper.
 * codes / What / prer as in oracle_quantize_layer_ex (original column order; What, prer may be NULL). */
int oracle_quantize_rows_factor(const float *W, int rows, int cols, int64_t ldw, const double *U,
                                const int32_t *perm, const float *scale, const float *zero, int bits,
                                uint8_t *codes, float *What, double *prer) {
    if (!W || !U || !perm || !scale || !zero || !codes || rows < 1 || cols < 1 || ldw < cols || bits < 2 ||
        bits > 8)
        return ORACLE_ERR_INVALID_ARG;
    const size_t n = (size_t)cols;
    const int maxq = (1 << bits) - 1;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < rows; ++i) {
        double *w = (double *)malloc(n * sizeof(double));
        if (!w) {
#pragma omp atomic write
            fail = 1;
            continue;
        }
        const double sc = (double)scale[i], zp = (double)zero[i];
        for (size_t p = 0; p < n; ++p) w[p] = (double)W[(size_t)i * (size_t)ldw + (size_t)perm[p]];
        for (size_t p = 0; p < n; ++p) {
            const double *Up = U + p * n;
            const size_t j0 = (size_t)perm[p];
            if (prer) prer[(size_t)i * n + j0] = w[p] / sc;
            const int c = quant_code(w[p], sc, zp, maxq);
            const double q = dequant(c, sc, zp);
            const double e = (w[p] - q) / Up[p];
            for (size_t j = p + 1; j < n; ++j) w[j] -= e * Up[j];
            codes[(size_t)i * n + j0] = (uint8_t)c;
            if (What) What[(size_t)i * n + j0] = (float)q;
        }
        free(w);
    }
    return fail ? ORACLE_ERR_NOMEM : ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Dynamic re-ranking (Sec. 5 writes the sort inside the per-column loop; read literally, the
 * columns still to be quantized are ranked again as the loop proceeds).  Every `block` columns
 * the scores of the REMAINING columns are recomputed from the CURRENT (compensated) weights and
 * the diagonal of the CURRENT (Eq.-12-updated) inverse Hessian, the remaining columns are sorted
 * by them (same keys, direction and tie rule as oracle_sensitivity_order), and the next `block`
 * columns are quantized in that order with Eq. 11 / Eq. 12 applied literally, in the original
 * index space (no permutation of A is ever formed).  block >= cols is the static method.
 *   order_out [cols]: the sequence in which the columns were quantized.
 * ------------------------------------------------------------------------------------- */
int oracle_quantize_layer_dynamic(const float *W, int rows, int cols, int64_t ldw, const double *Hinv,
                                  const float *scale, const float *zero, int bits, int mode_and_direction,
                                  int block, uint8_t *codes, float *What, int32_t *order_out,
                                  const double *H_undamped, double *loss_out, double *prer) {
    if (!W || !Hinv || !scale || !zero || !codes || !order_out || rows < 1 || cols < 1 || ldw < cols ||
        bits < 2 || bits > 8 || block < 1)
        return ORACLE_ERR_INVALID_ARG;
    const int ascending = (mode_and_direction & SCORE_ASCENDING) != 0;
    const int mode = mode_and_direction & ~SCORE_ASCENDING;
    if (mode < 0 || mode > SCORE_NONE) return ORACLE_ERR_INVALID_ARG;
    const size_t n = (size_t)cols, m = (size_t)rows;
    const int maxq = (1 << bits) - 1;
    double *A = (double *)malloc(n * n * sizeof(double));
    double *Wc = (double *)malloc(m * n * sizeof(double));
    double *S = (double *)malloc(n * sizeof(double));
    double *tcol = (double *)malloc(n * sizeof(double));
    int32_t *rest = (int32_t *)malloc(n * sizeof(int32_t));
    uint8_t *done = (uint8_t *)calloc(n, 1);
    if (!A || !Wc || !S || !tcol || !rest || !done) {
        free(A); free(Wc); free(S); free(tcol); free(rest); free(done);
        return ORACLE_ERR_NOMEM;
    }
    memcpy(A, Hinv, n * n * sizeof(double));
    for (size_t i = 0; i < m; ++i)
        for (size_t j = 0; j < n; ++j) Wc[i * n + j] = (double)W[i * (size_t)ldw + j];

    int status = ORACLE_OK;
    size_t count = 0;
    while (count < n && status == ORACLE_OK) {
        /* scores of the remaining columns, from the current weights and the current diagonal */
        size_t nrest = 0;
        for (size_t j = 0; j < n; ++j) {
            if (done[j]) continue;
            double s = 0.0;
            if (mode != SCORE_NONE) {
                for (size_t i = 0; i < m; ++i) {
                    const double w = Wc[i * n + j];
                    double num;
                    if (mode == SCORE_QERR || mode == SCORE_ERR) {
                        const double sc = (double)scale[i], zp = (double)zero[i];
                        const double q = dequant(quant_code(w, sc, zp, maxq), sc, zp);
                        num = (w - q) * (w - q);
                    } else {
                        num = w * w;
                    }
                    if (mode == SCORE_QERR || mode == SCORE_PRUNE) s += num / (2.0 * A[j * n + j]);
                    else s += num;
                }
            }
            if (!isfinite(s)) { status = ORACLE_ERR_INVALID_ARG; break; }
            S[j] = s;
            rest[nrest++] = (int32_t)j;
        }
        if (status != ORACLE_OK) break;
        g_sort_keys = S;
        g_sort_ascending = ascending;
        qsort(rest, nrest, sizeof(int32_t), cmp_score_stable);
        const size_t take = nrest < (size_t)block ? nrest : (size_t)block;
        for (size_t t = 0; t < take; ++t) {
            const size_t p = (size_t)rest[t];
            const double d = A[p * n + p];
            if (!(d > 0.0) || !isfinite(d)) { status = ORACLE_ERR_NOT_SPD; break; }
            const double *Ap = A + p * n;
#pragma omp parallel for schedule(static)
            for (size_t i = 0; i < m; ++i) {
                double *w = Wc + i * n;
                const double sc = (double)scale[i], zp = (double)zero[i];
                if (prer) prer[i * n + p] = w[p] / sc;
                const int c = quant_code(w[p], sc, zp, maxq);
                const double q = dequant(c, sc, zp);
                const double ei = (w[p] - q) / d;
                for (size_t j = 0; j < n; ++j)
                    if (!done[j] && j != p) w[j] -= ei * Ap[j]; /* Eq. 11 */
                w[p] = q;
                codes[i * n + p] = (uint8_t)c;
            }
            for (size_t j = 0; j < n; ++j) tcol[j] = A[j * n + p] / d;
#pragma omp parallel for schedule(static)
            for (size_t j = 0; j < n; ++j) { /* Eq. 12 on the columns still to come */
                if (done[j] || j == p) continue;
                double *Aj = A + j * n;
                const double tj = tcol[j];
                for (size_t k = 0; k < n; ++k)
                    if (!done[k] && k != p) Aj[k] -= tj * Ap[k];
            }
            for (size_t j = 0; j < n; ++j) { A[p * n + j] = 0.0; A[j * n + p] = 0.0; }
            done[p] = 1;
            order_out[count++] = (int32_t)p;
        }
    }
    if (status == ORACLE_OK) {
        if (What)
            for (size_t i = 0; i < m; ++i)
                for (size_t j = 0; j < n; ++j) What[i * n + j] = (float)Wc[i * n + j];
        if (H_undamped && loss_out) {
            double total = 0.0;
            for (size_t i = 0; i < m; ++i) {
                double acc = 0.0;
                for (size_t a = 0; a < n; ++a) {
                    const double da = (double)W[i * (size_t)ldw + a] - (double)(float)Wc[i * n + a];
                    double t = 0.0;
                    for (size_t b = 0; b < n; ++b)
                        t += H_undamped[a * n + b] * ((double)W[i * (size_t)ldw + b] - (double)(float)Wc[i * n + b]);
                    acc += da * t;
                }
                total += 0.5 * acc;
            }
            *loss_out = total;
        }
    }
    free(A); free(Wc); free(S); free(tcol); free(rest); free(done);
    return status;
}

/* ---------------------------------------------------------------------------------------
 * The non-parallel arm of the paper's ablation (Sec. 4.2, the paragraph on the per-row inverse
 * Hessians; the rows of Table 3 without the parallel tick): every row is ranked and quantized on
 * its own.  Row i sorts ITS weights by their own sensitivities L_ij (Sec. 4.1; the keys and tie
 * rule of oracle_sensitivity_order applied to that single row) and runs the column loop in that
 * order against a private copy of the inverse Hessian -- the [d_row, d_col, d_col] tensor, here
 * one slice at a time.  Cost rows * cols^3 / 3: small layers only.
 *   perm_rows [rows x cols]: the order each row used.
 * ------------------------------------------------------------------------------------- */
int oracle_quantize_layer_per_row(const float *W, int rows, int cols, int64_t ldw, const double *Hinv,
                                  const double *Hinv_diag, const float *scale, const float *zero, int bits,
                                  int mode_and_direction, uint8_t *codes, float *What, int32_t *perm_rows,
                                  const double *H_undamped, double *loss_out) {
    if (!W || !Hinv || !scale || !zero || !codes || !perm_rows || rows < 1 || cols < 1 || ldw < cols)
        return ORACLE_ERR_INVALID_ARG;
    const size_t n = (size_t)cols;
    double *S = (double *)malloc(n * sizeof(double));
    if (!S) return ORACLE_ERR_NOMEM;
    double total = 0.0;
    int status = ORACLE_OK;
    for (int i = 0; i < rows && status == ORACLE_OK; ++i) {
        const float *wi = W + (size_t)i * (size_t)ldw;
        int32_t *perm = perm_rows + (size_t)i * n;
        status = oracle_sensitivity_order(wi, 1, cols, ldw, Hinv_diag, scale + i, zero + i, bits,
                                          mode_and_direction, S, perm);
        if (status != ORACLE_OK) break;
        double loss = 0.0;
        status = oracle_quantize_layer_ex(wi, 1, cols, ldw, Hinv, perm, scale + i, zero + i, bits,
                                          codes + (size_t)i * n, What ? What + (size_t)i * n : NULL, H_undamped,
                                          H_undamped ? &loss : NULL, NULL, NULL, NULL, NULL, NULL);
        total += loss;
    }
    if (status == ORACLE_OK && H_undamped && loss_out) *loss_out = total;
    free(S);
    return status;
}
