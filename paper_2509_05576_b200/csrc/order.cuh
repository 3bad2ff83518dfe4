// Grid helper, column sensitivity scores and the stable descending column order (Sec. 4.2 steps 1-3).
#pragma once
#include "common.cuh"

namespace ptq {

// quant(): nearest level of the per-row grid, ties to even, clamped to the code range (all in float64).
__device__ __forceinline__ double quant_code_d(double w, double sc, double zp, double maxq) {
    double c = rint(w / sc) + zp;
    c = fmax(c, 0.0);
    c = fmin(c, maxq);
    return c;
}

// One CTA per row: lo = min(min_j w, 0), hi = max(max_j w, 0); scale = (hi - lo) / (2^bits - 1); zero = rint(-lo / scale).
__global__ void __launch_bounds__(256) minmax_grid_kernel(const float* __restrict__ W, int rows, int cols, int64_t ldw,
                                                           int bits, float* __restrict__ scale,
                                                           float* __restrict__ zero, int32_t* status) {
    __shared__ float slo[256], shi[256];
    __shared__ int sbad;
    const int i = blockIdx.x;
    if (threadIdx.x == 0) sbad = 0;
    __syncthreads();
    float lo = 0.f, hi = 0.f;
    bool bad = false;
    for (int j = threadIdx.x; j < cols; j += 256) {
        const float w = W[(int64_t)i * ldw + j];
        if (!isfinite(w)) bad = true;
        lo = fminf(lo, w);
        hi = fmaxf(hi, w);
    }
    if (bad) sbad = 1;
    slo[threadIdx.x] = lo;
    shi[threadIdx.x] = hi;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if (threadIdx.x < s) {
            slo[threadIdx.x] = fminf(slo[threadIdx.x], slo[threadIdx.x + s]);
            shi[threadIdx.x] = fmaxf(shi[threadIdx.x], shi[threadIdx.x + s]);
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        if (sbad) report(status, PTQ_ERR_NONFINITE, i);
        const double l = (double)slo[0], h = (double)shi[0];
        if (h == l) {
            scale[i] = 1.0f;
            zero[i] = 0.0f;
        } else {
            const double s = (h - l) / (double)((1 << bits) - 1);
            scale[i] = (float)s;
            zero[i] = (float)rint(-l / s);
        }
    }
}

constexpr int kScoreRowChunk = 64;

// partial[ch][j] = sum over the rows of chunk ch of the score numerator of w_ij.  T = float for the original weights,
// double for the compensated weights that dynamic re-ranking scores.
// One CTA per 64-row chunk and 32 columns: thread (g, c) adds rows 8 g .. 8 g + 7 of column c in ascending order (eight
// independent loads in flight), then the eight sub-sums of a column are added in ascending g: a fixed order, so the
// result does not depend on the launch.
constexpr int kScoreCols = 32;
template <typename T>
__global__ void __launch_bounds__(256) score_partial_kernel(const T* __restrict__ W, int rows, int cols,
                                                             int64_t ldw, const float* __restrict__ scale,
                                                             const float* __restrict__ zero, int bits, int mode,
                                                             double* __restrict__ partial) {
    __shared__ double sub[8][kScoreCols + 1];
    const int c = threadIdx.x & (kScoreCols - 1), g = threadIdx.x / kScoreCols;
    const int j = blockIdx.x * kScoreCols + c;
    const int ch = blockIdx.y;
    const int r0 = ch * kScoreRowChunk + g * (kScoreRowChunk / 8);
    const double maxq = (double)((1 << bits) - 1);
    const bool use_err = (mode == PTQ_SCORE_QERR || mode == PTQ_SCORE_ERR);
    double s = 0.0;
    if (j < cols) {
        double w[kScoreRowChunk / 8];
#pragma unroll
        for (int k = 0; k < kScoreRowChunk / 8; ++k) w[k] = r0 + k < rows ? (double)W[(int64_t)(r0 + k) * ldw + j] : 0.0;
#pragma unroll
        for (int k = 0; k < kScoreRowChunk / 8; ++k) {
            if (r0 + k >= rows) break;
            if (use_err) {
                const double sc = (double)scale[r0 + k], zp = (double)zero[r0 + k];
                const double q = sc * (quant_code_d(w[k], sc, zp, maxq) - zp);
                const double d = w[k] - q;
                s = fma(d, d, s);
            } else {
                s = fma(w[k], w[k], s);
            }
        }
    }
    sub[g][c] = s;
    __syncthreads();
    if (g == 0 && j < cols) {
        double t = sub[0][c];
#pragma unroll
        for (int k = 1; k < 8; ++k) t += sub[k][c];
        partial[(int64_t)ch * cols + j] = t;
    }
}

// S_j = (sum of the chunk partials, ascending) / (2 [Hinv]_jj)  for the sensitivity modes.
__global__ void __launch_bounds__(128) score_final_kernel(const double* __restrict__ partial, int chunks, int cols,
                                                           const double* __restrict__ hinv_diag, int mode,
                                                           double* __restrict__ S, int32_t* status) {
    const int j = blockIdx.x * 128 + threadIdx.x;
    if (j >= cols) return;
    double s = 0.0;
    if (mode != PTQ_SCORE_NONE) {
        for (int ch = 0; ch < chunks; ++ch) s += partial[(int64_t)ch * cols + j];
        if (mode == PTQ_SCORE_QERR || mode == PTQ_SCORE_PRUNE) s = s / (2.0 * hinv_diag[j]);
    }
    if (!isfinite(s)) report(status, PTQ_ERR_NONFINITE, j);
    S[j] = s;
}

// Order-preserving map from float64 to uint64 (total order, so even non-finite scores give a permutation).
__device__ __forceinline__ unsigned long long sortable_key(double x) {
    unsigned long long u = (unsigned long long)__double_as_longlong(x);
    return (u & 0x8000000000000000ull) ? ~u : (u | 0x8000000000000000ull);
}

// perm[rank_j] = j with rank_j = #{k : S_k > S_j, or S_k == S_j and k < j}: a stable descending sort by counting
// (ascending != 0: S_k < S_j instead, the "asc" keys of Sec. 4.1; equal scores keep the lower index first either way).
// 16 columns j per CTA; the 16 lanes that share a column each count a strided sixteenth of the keys, which are staged in
// shared memory 2048 at a time.  A chunk is padded to a multiple of 128 keys with entries that never count (key 0 with
// the largest tie value), so the counting loop runs in unrolled groups of eight without a bound test.
constexpr int kRankCols = 16;
constexpr int kRankChunk = 2048;
// tie != nullptr: equal scores are ordered by tie[] (distinct values) instead of by position.
__global__ void __launch_bounds__(256) rank_sort_kernel(const double* __restrict__ S, int cols, int ascending,
                                                         int32_t* __restrict__ perm,
                                                         const int32_t* __restrict__ tie = nullptr) {
    __shared__ unsigned long long keys[kRankChunk];
    __shared__ int32_t ties[kRankChunk];
    const int j = blockIdx.x * kRankCols + (threadIdx.x >> 4);
    const int part = threadIdx.x & 15;
    // ascending order is descending order of the complemented keys
    const unsigned long long flip = ascending ? ~0ull : 0ull;
    const unsigned long long kj = j < cols ? (sortable_key(S[j]) ^ flip) : 0ull;
    const int tj = (tie != nullptr && j < cols) ? tie[j] : j;
    int rank = 0;
    for (int t0 = 0; t0 < cols; t0 += kRankChunk) {
        const int lim = min(kRankChunk, cols - t0);
        const int lim_pad = (lim + 127) & ~127;
        for (int t = threadIdx.x; t < lim_pad; t += 256) {
            const bool in = t < lim;
            keys[t] = in ? (sortable_key(S[t0 + t]) ^ flip) : 0ull;
            ties[t] = in ? (tie != nullptr ? tie[t0 + t] : t0 + t) : 0x7fffffff;
        }
        __syncthreads();
        for (int base = part; base < lim_pad; base += 128) {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const unsigned long long kk = keys[base + 16 * u];
                const int tt = ties[base + 16 * u];
                rank += (kk > kj || (kk == kj && tt < tj)) ? 1 : 0;
            }
        }
        __syncthreads();
    }
    rank += __shfl_xor_sync(0xffffffffu, rank, 1);
    rank += __shfl_xor_sync(0xffffffffu, rank, 2);
    rank += __shfl_xor_sync(0xffffffffu, rank, 4);
    rank += __shfl_xor_sync(0xffffffffu, rank, 8);
    if (part == 0 && j < cols) perm[rank] = j;
}

}  // namespace ptq
