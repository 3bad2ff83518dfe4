// Dynamic re-ranking (Sec. 5 places the sort inside the per-column loop): the columns still to be quantized are ranked
// again every `block` columns, from the compensated weights and the diagonal of the Eq.-12-updated inverse Hessian.
//
// One round, with m columns left, A the current m x m matrix (what Eq. 12 has left of the inverse Hessian) and Wc the
// current weights: scores and order of the m columns; both are gathered into that order; the first b = min(block, m)
// block rows of the Cholesky factor of A are computed, which leaves the Schur complement of the leading b x b block --
// the matrix Eq. 12 leaves after those b columns -- in the rest; the first b columns are swept with those rows of the
// factor; the remaining columns absorb the b columns' errors in one product, Wc[:, b:] -= E U[:b, b:] (Eq. 11, deferred).
// The rest of A and Wc are the next round's inputs.  Only the upper triangle of A is kept up to date.
#pragma once
#include "common.cuh"
#include "order.cuh"

namespace ptq {

__global__ void iota_kernel(int32_t* __restrict__ a, int n) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < n) a[j] = j;
}

__global__ void extract_diag_ld_kernel(const double* __restrict__ A, int64_t ld, int m, double* __restrict__ d) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < m) d[j] = A[(int64_t)j * ld + j];
}

// Anew[a][c] = A[lo][hi] with {lo, hi} = {ordr[a], ordr[c]} sorted: reads the upper triangle of A only.  One CTA row per a.
__global__ void gather_upper_kernel(const double* __restrict__ A, int64_t ld, const int32_t* __restrict__ ordr, int m,
                                    double* __restrict__ Anew) {
    for (int a = blockIdx.y; a < m; a += gridDim.y) {
        const int oa = ordr[a];
        for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < m; c += gridDim.x * blockDim.x) {
            const int oc = ordr[c];
            const int lo = oa < oc ? oa : oc, hi = oa < oc ? oc : oa;
            Anew[(int64_t)a * m + c] = A[(int64_t)lo * ld + hi];
        }
    }
}

// Wnew[i][p] = (double) Wc[i][ordr[p]]
template <typename T>
__global__ void gather_cols_kernel(const T* __restrict__ Wc, int64_t ld, int rows, int m,
                                   const int32_t* __restrict__ ordr, double* __restrict__ Wnew) {
    for (int i = blockIdx.y; i < rows; i += gridDim.y)
        for (int p = blockIdx.x * blockDim.x + threadIdx.x; p < m; p += gridDim.x * blockDim.x)
            Wnew[(int64_t)i * m + p] = (double)Wc[(int64_t)i * ld + ordr[p]];
}

// orig_new[p] = orig[ordr[p]]: original column index of the column now at position p; the first b go to order_out.
__global__ void gather_index_kernel(const int32_t* __restrict__ orig, const int32_t* __restrict__ ordr, int m, int b,
                                    int32_t* __restrict__ orig_new, int32_t* __restrict__ order_out) {
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= m) return;
    const int o = orig[ordr[p]];
    orig_new[p] = o;
    if (p < b) order_out[p] = o;
}

// The b columns just swept go out in the ORIGINAL column order: codes, What = float32(scale (code - zero)), dW = W - What.
__global__ void emit_block_kernel(const uint8_t* __restrict__ codes_p, int64_t ld, const int32_t* __restrict__ orig, int b,
                                  const float* __restrict__ W, int rows, int cols, int64_t ldw,
                                  const float* __restrict__ scale, const float* __restrict__ zero,
                                  uint8_t* __restrict__ codes, float* __restrict__ What, double* __restrict__ dW) {
    for (int i = blockIdx.y; i < rows; i += gridDim.y) {
        const double sc = (double)scale[i], zp = (double)zero[i];
        for (int p = blockIdx.x * blockDim.x + threadIdx.x; p < b; p += gridDim.x * blockDim.x) {
            const int j = orig[p];
            const uint8_t c = codes_p[(int64_t)i * ld + p];
            codes[(int64_t)i * cols + j] = c;
            const float q = (float)(sc * ((double)c - zp));
            if (What) What[(int64_t)i * cols + j] = q;
            if (dW) dW[(int64_t)i * cols + j] = (double)W[(int64_t)i * ldw + j] - (double)q;
        }
    }
}

}  // namespace ptq
