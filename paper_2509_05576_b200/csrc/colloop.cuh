// The column-synchronous quantization sweep (Sec. 4.2 steps 3-5, Eq. 11 / Eq. 12) in blocked form.
//
// With A the permuted inverse Hessian and A = U^T U its upper Cholesky factor, the matrix that Eq. 12 leaves
// before step p has row p equal to sqrt(pivot) * U[p, p:], so Eq. 11 for column p reads
//     e_i = (w_ip - q_ip) / U[p][p],      w_ij -= e_i * U[p][j]   for j > p.
// Columns are processed in blocks of 64: inside a block every row is swept by one thread that keeps the
// block's 64 weights in registers; the effect of the block on all later columns is one float64 GEMM,
// W[:, later] -= E[:, block] U[block, later].
#pragma once
#include "common.cuh"
#include "dgemm.cuh"
#include "order.cuh"

namespace ptq {

// flags[] must be zero on entry.  Reports out-of-range or repeated entries; invperm[perm[p]] = p.
__global__ void perm_check_kernel(const int32_t* __restrict__ perm, int cols, int32_t* __restrict__ flags,
                                  int32_t* __restrict__ invperm, int32_t* status) {
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= cols) return;
    const int j = perm[p];
    if (j < 0 || j >= cols) { report(status, PTQ_ERR_INVALID_ARG, p, 1); return; }
    if (atomicExch(&flags[j], 1) != 0) { report(status, PTQ_ERR_INVALID_ARG, p, 2); return; }
    invperm[j] = p;
}

__device__ __forceinline__ int clamp_index(int j, int n) { return j < 0 ? 0 : (j >= n ? n - 1 : j); }

// A[a][b] = Hinv[perm[a]][perm[b]]
__global__ void gather_sym_kernel(const double* __restrict__ Hinv, const int32_t* __restrict__ perm, int n,
                                  double* __restrict__ A) {
    const int a = blockIdx.y;
    const int64_t src = (int64_t)clamp_index(perm[a], n) * n;
    for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < n; b += gridDim.x * blockDim.x)
        A[(int64_t)a * n + b] = Hinv[src + clamp_index(perm[b], n)];
}

// Wp[i][p] = (double) W[i][perm[p]]
__global__ void gather_w_kernel(const float* __restrict__ W, int rows, int cols, int64_t ldw,
                                const int32_t* __restrict__ perm, double* __restrict__ Wp) {
    const int i = blockIdx.y;
    for (int p = blockIdx.x * blockDim.x + threadIdx.x; p < cols; p += gridDim.x * blockDim.x)
        Wp[(int64_t)i * cols + p] = (double)W[(int64_t)i * ldw + clamp_index(perm[p], cols)];
}

constexpr int kRowsPerCta = 32;
constexpr size_t kColloopSmem =
    sizeof(double) * (kNB * kNB + kRowsPerCta * (kNB + 1) + kNB) + kRowsPerCta * (kNB + 4);

// One block of 64 columns starting at p0, 32 rows per CTA.  All 128 threads stage the tile; warp 0 runs the
// dependent chain, one row per lane.  Outputs: E[:, p0:p0+kb] (scaled errors) and codes (permuted order).
__global__ void __launch_bounds__(128) colloop_block_kernel(const double* __restrict__ Wp, int rows, int cols,
                                                             int p0, int kb, const double* __restrict__ U,
                                                             const float* __restrict__ scale,
                                                             const float* __restrict__ zero, int bits,
                                                             double* __restrict__ E, uint8_t* __restrict__ codes_p) {
    extern __shared__ __align__(16) unsigned char colloop_smem[];
    double (*Us)[kNB] = reinterpret_cast<double (*)[kNB]>(colloop_smem);
    double (*Ws)[kNB + 1] = reinterpret_cast<double (*)[kNB + 1]>(colloop_smem + sizeof(double) * kNB * kNB);
    double* rdiag = reinterpret_cast<double*>(colloop_smem + sizeof(double) * (kNB * kNB + kRowsPerCta * (kNB + 1)));
    uint8_t (*Cs)[kNB + 4] = reinterpret_cast<uint8_t (*)[kNB + 4]>(
        colloop_smem + sizeof(double) * (kNB * kNB + kRowsPerCta * (kNB + 1) + kNB));
    const int tid = threadIdx.x;
    const int row0 = blockIdx.x * kRowsPerCta;

    for (int idx = tid; idx < kNB * kNB; idx += 128) {
        const int r = idx >> 6, c = idx & 63;
        double v = (r == c) ? 1.0 : 0.0;
        if (r < kb && c < kb && c >= r) v = U[(int64_t)(p0 + r) * cols + p0 + c];
        Us[r][c] = v;
    }
    for (int idx = tid; idx < kRowsPerCta * kNB; idx += 128) {
        const int r = idx >> 6, c = idx & 63;
        double v = 0.0;
        if (row0 + r < rows && c < kb) v = Wp[(int64_t)(row0 + r) * cols + p0 + c];
        Ws[r][c] = v;
    }
    __syncthreads();
    if (tid < kNB) rdiag[tid] = 1.0 / Us[tid][tid];
    __syncthreads();

    if (tid < 32) {
        const int row = row0 + tid;
        const bool live = row < rows;
        const double sc = live ? (double)scale[row] : 1.0;
        const double zp = live ? (double)zero[row] : 0.0;
        const double maxq = (double)((1 << bits) - 1);
        double w[kNB];
#pragma unroll
        for (int c = 0; c < kNB; ++c) w[c] = Ws[tid][c];
#pragma unroll
        for (int p = 0; p < kNB; ++p) {
            const double c = quant_code_d(w[p], sc, zp, maxq);
            const double q = sc * (c - zp);
            const double e = (w[p] - q) * rdiag[p];
#pragma unroll
            for (int j = p + 1; j < kNB; ++j) w[j] = fma(-e, Us[p][j], w[j]);
            Ws[tid][p] = e;
            Cs[tid][p] = (uint8_t)(int)c;
        }
    }
    __syncthreads();
    for (int idx = tid; idx < kRowsPerCta * kNB; idx += 128) {
        const int r = idx >> 6, c = idx & 63;
        if (row0 + r < rows && c < kb) {
            E[(int64_t)(row0 + r) * cols + p0 + c] = Ws[r][c];
            codes_p[(int64_t)(row0 + r) * cols + p0 + c] = Cs[r][c];
        }
    }
}

// Back to the original column order: codes, What = float32(scale * (code - zero)), dW = W - What (float64).
__global__ void finalize_kernel(const uint8_t* __restrict__ codes_p, const int32_t* __restrict__ invperm,
                                const float* __restrict__ W, int rows, int cols, int64_t ldw,
                                const float* __restrict__ scale, const float* __restrict__ zero,
                                uint8_t* __restrict__ codes, float* __restrict__ What, double* __restrict__ dW) {
    const int i = blockIdx.y;
    const double sc = (double)scale[i], zp = (double)zero[i];
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < cols; j += gridDim.x * blockDim.x) {
        const uint8_t c = codes_p[(int64_t)i * cols + invperm[j]];
        codes[(int64_t)i * cols + j] = c;
        const float q = (float)(sc * ((double)c - zp));
        if (What) What[(int64_t)i * cols + j] = q;
        if (dW) dW[(int64_t)i * cols + j] = (double)W[(int64_t)i * ldw + j] - (double)q;
    }
}

// out = factor * (sum of partials in a fixed order)
__global__ void __launch_bounds__(256) sum_partials_kernel(const double* __restrict__ partials, int count,
                                                            double factor, double* __restrict__ out) {
    __shared__ double red[256];
    double s = 0.0;
    for (int k = threadIdx.x; k < count; k += 256) s += partials[k];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = factor * red[0];
}

}  // namespace ptq
