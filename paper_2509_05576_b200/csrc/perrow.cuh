// The non-parallel arm of the paper's ablation (Sec. 4.2, the paragraph on the per-row inverse Hessians; the rows of
// Table 3 without the parallel tick): every row ranks ITS weights by their own sensitivities (Sec. 4.1) and is quantized
// in that order against a private copy of the inverse Hessian -- the [d_row, d_col, d_col] tensor, one slice per CTA,
// held in shared memory.  Cost rows * cols^3 / 3, which is what the row-parallel method saves; narrow layers only.
#pragma once
#include "common.cuh"
#include "order.cuh"

namespace ptq {

constexpr int kPerRowMaxCols = 128;
constexpr int kPerRowThreads = 256;
inline size_t per_row_smem_bytes(int cols) {
    return sizeof(double) * ((size_t)cols * (cols + 1) + 3 * (size_t)cols) + sizeof(int32_t) * (size_t)cols + 64;
}

// One CTA per row i.
//   1. L_j = score of w_ij (the keys of ptq_sensitivity_order on this single row); perm = stable sort of the columns
//   2. A = Hinv[perm][:, perm] in shared memory; A = U^T U by a right-looking Cholesky (one barrier per pivot: the
//      pivot row stays unscaled while it is in use and all rows are scaled by 1 / sqrt(pivot) at the end)
//   3. the column loop on the row: c = quant(w_p), e = (w_p - q) / U_pp, w_j -= e U_pj (Eq. 11 with the row of the
//      Eq.-12-updated matrix written through the factor)
//   4. codes, What and the order go out; row_loss[i] = 1/2 dw H dw^T
__global__ void __launch_bounds__(kPerRowThreads) per_row_kernel(const float* __restrict__ W, int rows, int cols, int64_t ldw,
                                                                 const double* __restrict__ Hinv,
                                                                 const float* __restrict__ scale,
                                                                 const float* __restrict__ zero, int bits, int mode,
                                                                 int ascending, uint8_t* __restrict__ codes,
                                                                 float* __restrict__ What, int32_t* __restrict__ perm_rows,
                                                                 const double* __restrict__ H, double* __restrict__ row_loss,
                                                                 int32_t* status) {
    extern __shared__ __align__(16) unsigned char per_row_smem[];
    const int n = cols, lda = cols + 1;
    double* A = reinterpret_cast<double*>(per_row_smem);          // [n][n + 1]
    double* w = A + (size_t)n * lda;                               // [n] weights in the row's own order
    double* key = w + n;                                           // [n] scores, later 1 / sqrt(pivot)
    double* dw = key + n;                                          // [n] w - What, original order
    int32_t* perm = reinterpret_cast<int32_t*>(dw + n);            // [n]
    __shared__ double red[kPerRowThreads];
    const int i = blockIdx.x, tid = threadIdx.x;
    const double sc = (double)scale[i], zp = (double)zero[i];
    const double maxq = (double)((1 << bits) - 1);

    // 1. scores and order
    for (int j = tid; j < n; j += kPerRowThreads) {
        const double x = (double)W[(int64_t)i * ldw + j];
        double num = 0.0;
        if (mode == PTQ_SCORE_QERR || mode == PTQ_SCORE_ERR) {
            const double d = x - sc * (quant_code_d(x, sc, zp, maxq) - zp);
            num = d * d;
        } else if (mode == PTQ_SCORE_PRUNE || mode == PTQ_SCORE_W) {
            num = x * x;
        }
        if (mode == PTQ_SCORE_QERR || mode == PTQ_SCORE_PRUNE) num = num / (2.0 * Hinv[(int64_t)j * n + j]);
        key[j] = num;
    }
    __syncthreads();
    for (int j = tid; j < n; j += kPerRowThreads) {
        const unsigned long long flip = ascending ? ~0ull : 0ull;
        const unsigned long long kj = sortable_key(key[j]) ^ flip;
        int rank = 0;
        for (int t = 0; t < n; ++t) {
            const unsigned long long kt = sortable_key(key[t]) ^ flip;
            rank += (kt > kj || (kt == kj && t < j)) ? 1 : 0;
        }
        perm[rank] = j;
    }
    __syncthreads();
    // 2. the row's own permuted inverse Hessian (upper triangle) and its factor
    for (int idx = tid; idx < n * n; idx += kPerRowThreads) {
        const int a = idx / n, c = idx - a * n;
        if (c >= a) A[a * lda + c] = Hinv[(int64_t)perm[a] * n + perm[c]];
    }
    for (int p = tid; p < n; p += kPerRowThreads) w[p] = (double)W[(int64_t)i * ldw + perm[p]];
    const int lane = tid & 31, warp = tid >> 5;
    for (int p = 0; p < n; ++p) {
        __syncthreads();
        const double d0 = A[p * lda + p];
        const bool ok = d0 > 0.0 && d0 < 1.0e300;
        if (!ok && tid == 0) report(status, PTQ_ERR_NOT_SPD, p, i);
        const double inv = 1.0 / (ok ? d0 : 1.0);
        const double* rp = A + p * lda;
        for (int r = p + 1 + warp; r < n; r += kPerRowThreads / 32) {
            const double f = rp[r] * inv;
            double* rr = A + r * lda;
            for (int c = r + lane; c < n; c += 32) rr[c] = fma(-f, rp[c], rr[c]);
        }
    }
    __syncthreads();
    for (int p = tid; p < n; p += kPerRowThreads) {
        const double d0 = A[p * lda + p];
        key[p] = rsqrt(d0 > 0.0 && d0 < 1.0e300 ? d0 : 1.0);
    }
    __syncthreads();
    for (int idx = tid; idx < n * n; idx += kPerRowThreads) {
        const int a = idx / n, c = idx - a * n;
        if (c >= a) A[a * lda + c] *= key[a];
    }
    // 3. the column loop; every thread takes the (same) rounding decision itself, then updates its own columns
    for (int p = 0; p < n; ++p) {
        __syncthreads();
        const double x = w[p];
        const double cdec = quant_code_d(x, sc, zp, maxq);
        const double q = sc * (cdec - zp);
        const double e = (x - q) / A[p * lda + p];
        for (int c = p + 1 + tid; c < n; c += kPerRowThreads) w[c] = fma(-e, A[p * lda + c], w[c]);
        if (tid == 0) {
            const int j = perm[p];
            codes[(int64_t)i * n + j] = (uint8_t)(int)cdec;
            const float qf = (float)q;
            if (What) What[(int64_t)i * n + j] = qf;
            dw[j] = (double)W[(int64_t)i * ldw + j] - (double)qf;
        }
    }
    __syncthreads();
    for (int p = tid; p < n; p += kPerRowThreads) perm_rows[(int64_t)i * n + p] = perm[p];
    // 4. 1/2 dw H dw^T for this row
    if (H != nullptr && row_loss != nullptr) {
        double s = 0.0;
        for (int a = tid; a < n; a += kPerRowThreads) {
            double t = 0.0;
            for (int b = 0; b < n; ++b) t = fma(H[(int64_t)a * n + b], dw[b], t);
            s = fma(dw[a], t, s);
        }
        red[tid] = s;
        __syncthreads();
        for (int wd = kPerRowThreads / 2; wd > 0; wd >>= 1) {
            if (tid < wd) red[tid] += red[tid + wd];
            __syncthreads();
        }
        if (tid == 0) row_loss[i] = 0.5 * red[0];
    }
}

}  // namespace ptq
