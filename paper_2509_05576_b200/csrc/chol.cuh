// Float64 blocked factorisation pieces: A = U^T U (upper Cholesky, in place, row-major), the inverse of the
// factor by recursive halving, and Hinv = V V^T.  Sec. 5 item 1 of the paper (Cholesky, then the inverse of
// the factor); the same Cholesky applied to the permuted inverse Hessian is the blocked form of Eq. 12:
// step p of a right-looking Cholesky subtracts (row p)^T (row p) / pivot from the trailing matrix.
#pragma once
#include "common.cuh"
#include "dgemm.cuh"

namespace ptq {

// lambda = damp * mean(diag H) or damp; one CTA, fixed summation order.  Flags non-finite diagonals.
__global__ void __launch_bounds__(256) lambda_kernel(const double* __restrict__ H, int n, int mode, double damp,
                                                      double* __restrict__ lambda_out, int32_t* status) {
    __shared__ double red[256];
    double s = 0.0;
    bool bad = false;
    for (int j = threadIdx.x; j < n; j += 256) {
        const double d = H[(int64_t)j * n + j];
        if (!isfinite(d)) bad = true;
        s += d;
    }
    if (bad) report(status, PTQ_ERR_NONFINITE, -1);
    red[threadIdx.x] = s;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
        __syncthreads();
    }
    if (threadIdx.x == 0) *lambda_out = mode == PTQ_DAMP_REL_MEAN_DIAG ? damp * (red[0] / (double)n) : damp;
}

// A = H + lambda I
__global__ void damp_copy_kernel(const double* __restrict__ H, double* __restrict__ A, int n,
                                 const double* __restrict__ lambda) {
    const int64_t total = (int64_t)n * n;
    const double lam = *lambda;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int i = (int)(idx / n), j = (int)(idx - (int64_t)i * n);
        A[idx] = H[idx] + (i == j ? lam : 0.0);
    }
}

// Upper Cholesky of the kb x kb diagonal block at (k0, k0), one CTA.  Row p of the factor is written to
// global memory as soon as step p fixes it.  A non-positive or non-finite pivot is reported and replaced by 1.
__global__ void __launch_bounds__(256) potrf_diag_kernel(double* __restrict__ A, int64_t ld, int k0, int kb,
                                                          int32_t* status) {
    __shared__ double S[kNB][kNB + 1];
    const int tid = threadIdx.x;
    for (int idx = tid; idx < kNB * kNB; idx += 256) {
        const int r = idx >> 6, c = idx & 63;
        double v = (r == c) ? 1.0 : 0.0;
        if (r < kb && c < kb && c >= r) v = A[(int64_t)(k0 + r) * ld + k0 + c];
        S[r][c] = v;
    }
    __syncthreads();
    for (int p = 0; p < kNB; ++p) {
        double d = S[p][p];
        if (!(d > 0.0) || !isfinite(d)) {
            if (tid == 0) report(status, PTQ_ERR_NOT_SPD, k0 + p);
            d = 1.0;
        }
        const double inv = 1.0 / d;
        if (tid >= p && tid < kb && p < kb) A[(int64_t)(k0 + p) * ld + k0 + tid] = S[p][tid] / sqrt(d);
        for (int idx = tid; idx < kNB * kNB; idx += 256) {
            const int i = idx >> 6, j = idx & 63;
            if (i > p && j >= i) S[i][j] -= S[p][i] * S[p][j] * inv;
        }
        __syncthreads();
    }
}

// Row panel: U[k0:k0+kb, c] = U_kk^-T A[k0:k0+kb, c] for the columns c >= k0 + kb, one thread per column
// (forward substitution against the transposed diagonal factor held in shared memory).
__global__ void __launch_bounds__(128) panel_solve_kernel(double* __restrict__ A, int64_t ld, int k0, int kb, int n) {
    __shared__ double Us[kNB][kNB];
    for (int idx = threadIdx.x; idx < kNB * kNB; idx += 128) {
        const int r = idx >> 6, c = idx & 63;
        double v = (r == c) ? 1.0 : 0.0;
        if (r < kb && c < kb && c >= r) v = A[(int64_t)(k0 + r) * ld + k0 + c];
        Us[r][c] = v;
    }
    __syncthreads();
    const int col = k0 + kb + blockIdx.x * 128 + threadIdx.x;
    if (col >= n) return;
    double y[kNB];
#pragma unroll
    for (int r = 0; r < kNB; ++r) y[r] = (r < kb) ? A[(int64_t)(k0 + r) * ld + col] : 0.0;
#pragma unroll
    for (int r = 0; r < kNB; ++r) {
        double s = y[r];
#pragma unroll
        for (int t = 0; t < r; ++t) s = fma(-Us[t][r], y[t], s);
        y[r] = s / Us[r][r];
    }
#pragma unroll
    for (int r = 0; r < kNB; ++r)
        if (r < kb) A[(int64_t)(k0 + r) * ld + col] = y[r];
}

// In-place blocked upper Cholesky of the n x n matrix A (only the upper triangle is read or written as a result).
inline int cholesky_upper(double* A, int n, int32_t* status, cudaStream_t stream) {
    for (int k0 = 0; k0 < n; k0 += kNB) {
        const int kb = n - k0 < kNB ? n - k0 : kNB;
        { Launch l(K_POTRF_DIAG, stream); potrf_diag_kernel<<<1, 256, 0, stream>>>(A, n, k0, kb, status); }
        const int rest = n - k0 - kb;
        if (rest <= 0) break;
        { Launch l(K_PANEL_SOLVE, stream); panel_solve_kernel<<<cdiv(rest, 128), 128, 0, stream>>>(A, n, k0, kb, n); }
        GemmParams g = gemm_defaults();     // A22 -= U12^T U12 on the upper tiles
        g.A = A + (int64_t)k0 * n + k0 + kb; g.lda = n; g.a_trans = 1;
        g.B = g.A; g.ldb = n; g.b_trans = 0;
        g.C = A + (int64_t)(k0 + kb) * n + k0 + kb; g.ldc = n;
        g.M = rest; g.N = rest; g.K = kb;
        g.alpha = -1.0; g.beta = 1.0; g.upper_only = 1;
        int st = launch_dgemm(K_DGEMM_CHOL, g, 1, stream);
        if (st) return st;
    }
    return launch_status();
}

// V[b, b] = inverse of the upper-triangular diagonal block R[b, b]; one CTA per 64-block, one thread per column.
__global__ void __launch_bounds__(kNB) diag_inverse_kernel(const double* __restrict__ R, double* __restrict__ V,
                                                            int64_t ld, int n) {
    __shared__ double Us[kNB][kNB];
    const int b0 = blockIdx.x * kNB;
    const int kb = n - b0 < kNB ? n - b0 : kNB;
    for (int idx = threadIdx.x; idx < kNB * kNB; idx += kNB) {
        const int r = idx >> 6, c = idx & 63;
        double v = (r == c) ? 1.0 : 0.0;
        if (r < kb && c < kb && c >= r) v = R[(int64_t)(b0 + r) * ld + b0 + c];
        Us[r][c] = v;
    }
    __syncthreads();
    const int j = threadIdx.x;
    double v[kNB];
#pragma unroll
    for (int i = kNB - 1; i >= 0; --i) {
        double s = (i == j) ? 1.0 : 0.0;
#pragma unroll
        for (int k = i + 1; k < kNB; ++k) s = fma(-Us[i][k], v[k], s);
        v[i] = s / Us[i][i];
    }
    if (j < kb) {
#pragma unroll
        for (int i = 0; i < kNB; ++i)
            if (i <= j) V[(int64_t)(b0 + i) * ld + b0 + j] = v[i];
    }
}

// V = R^-1 for upper-triangular R (n x n).  V must be zero on entry; T is n x n scratch.
// Recursive halving: with R = [R11 R12; 0 R22], V12 = -V11 (R12 V22); all pairs of one level run as one batch.
inline int trtri_upper(const double* R, double* V, double* T, int n, cudaStream_t stream) {
    { Launch l(K_DIAG_INVERSE, stream); diag_inverse_kernel<<<cdiv(n, kNB), kNB, 0, stream>>>(R, V, n, n); }
    for (int64_t s = kNB; s < n; s *= 2) {
        const int pairs = (int)((n + 2 * s - 1) / (2 * s));
        const int64_t step = 2 * s * ((int64_t)n + 1);
        GemmParams g = gemm_defaults();     // T12 = R12 V22   (V22 upper: k stops at the tile's last column)
        g.A = R + s; g.lda = n; g.a_trans = 0; g.batch_a = step;
        g.B = V + s * ((int64_t)n + 1); g.ldb = n; g.b_trans = 0; g.batch_b = step;
        g.C = T + s; g.ldc = n; g.batch_c = step;
        g.M = (int)s; g.N = (int)s; g.K = (int)s;
        g.ragN_lim = n - (int)s; g.ragN_step = (int)(2 * s); g.k_is_n = 1;
        g.kend_mode = 1;
        int st = launch_dgemm(K_DGEMM_TRTRI, g, pairs, stream);
        if (st) return st;
        GemmParams h = gemm_defaults();     // V12 = -V11 T12   (V11 upper: k starts at the tile's first row)
        h.A = V; h.lda = n; h.a_trans = 0; h.batch_a = step;
        h.B = T + s; h.ldb = n; h.b_trans = 0; h.batch_b = step;
        h.C = V + s; h.ldc = n; h.batch_c = step;
        h.M = (int)s; h.N = (int)s; h.K = (int)s;
        h.ragN_lim = n - (int)s; h.ragN_step = (int)(2 * s);
        h.kbeg_mode = 2;
        h.alpha = -1.0;
        st = launch_dgemm(K_DGEMM_TRTRI, h, pairs, stream);
        if (st) return st;
    }
    return launch_status();
}

// Hinv = V V^T for upper-triangular V: the sum over k starts at max(i, j); upper tiles computed, mirrored below.
inline int lauum_upper(const double* V, double* Hinv, int n, cudaStream_t stream) {
    GemmParams g = gemm_defaults();
    g.A = V; g.lda = n; g.a_trans = 0;
    g.B = V; g.ldb = n; g.b_trans = 1;
    g.C = Hinv; g.ldc = n;
    g.M = n; g.N = n; g.K = n;
    g.kbeg_mode = 1; g.upper_only = 1; g.mirror = 1;
    return launch_dgemm(K_DGEMM_LAUUM, g, 1, stream);
}

__global__ void extract_diag_kernel(const double* __restrict__ A, int n, double* __restrict__ d) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < n) d[j] = A[(int64_t)j * n + j];
}

}  // namespace ptq
