// Float64 blocked factorisation pieces: A = U^T U (upper Cholesky, in place, row-major), the inverse of the
// factor by recursive halving, and Hinv = V V^T.  Sec. 5 item 1 of the paper (Cholesky, then the inverse of
// the factor); the same Cholesky applied to the permuted inverse Hessian is the blocked form of Eq. 12:
// step p of a right-looking Cholesky subtracts (row p)^T (row p) / pivot from the trailing matrix.
#pragma once
#include "common.cuh"
#include "dgemm.cuh"
#include <utility>

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

// ------------------------------------------------------------------------------------------------------------
// Blocked upper Cholesky A = U^T U as ONE persistent cooperative kernel (one CTA per SM, 256 threads).
// For each 64-row block k:
//   strip phase    every CTA that owns panel columns factorises the 64 x 64 diagonal block itself (all CTAs do the
//                  same arithmetic on it, so no broadcast is needed) and applies the same row operations to its own
//                  192 panel columns: one thread per column, the column's 64 entries in registers, row p of the
//                  diagonal block broadcast through shared memory at step p.  That is the unblocked algorithm on a
//                  64-row strip, and it replaces "factor the block, then solve the panel against it".
//   trailing phase A[i][j] -= U[k][i]^T U[k][j] on the upper 64 x 64 tiles, float64 tensor-core MMA, operands
//                  double-buffered through shared memory with cp.async.
// The phases are separated by a grid-wide barrier whose wait is bounded: when it expires the CTA records
// PTQ_ERR_TIMEOUT, raises the abort word and leaves; the other CTAs see the abort word and leave too.
// A non-positive or non-finite pivot is reported (PTQ_ERR_NOT_SPD, pivot index) and replaced by 1.
// ------------------------------------------------------------------------------------------------------------
constexpr int kCholThreads = 256;
constexpr int kCholPanelCols = kCholThreads - kNB;            // 192 panel columns per CTA in the strip phase
constexpr int kCholLd = kNB + 4;                               // operand row stride (68 = 4 mod 16: conflict-free)
constexpr size_t kCholSmemBytes = sizeof(double) * (2 * 2 * kNB * kCholLd + 2 * kNB) + 16;

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// bar[0]: arrival counter (monotonic, zero at launch), bar[1]: abort word.  Returns false when the CTA must leave.
__device__ __forceinline__ bool grid_barrier(unsigned* bar, unsigned target, int* s_flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(&bar[0], 1u);
        const long long t0 = clock64();
        int ok = 1;
        unsigned it = 0;
        while (ld_acquire_u32(&bar[0]) < target) {
            if ((++it & 63u) == 0u) {
                if (ld_acquire_u32(&bar[1]) != 0u) { ok = 0; break; }
                if (clock64() - t0 > 4000000000LL) { atomicExch(&bar[1], 1u); ok = 0; break; }
            }
        }
        __threadfence();
        *s_flag = ok;
    }
    __syncthreads();
    return *s_flag != 0;
}

__device__ __forceinline__ void cp_async16_cg(void* smem_dst, const void* gsrc, bool valid) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const int sz = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(gsrc), "r"(sz) : "memory");
}

// Loads the 64 x 64 block A[r0 .. r0+63][c0 .. c0+63] into dst[64][kCholLd]; entries beyond n are zero.
__device__ __forceinline__ void chol_load_block(double* dst, const double* __restrict__ A, int64_t ld, int n, int r0,
                                                int c0, int vec16) {
    if (vec16) {
        for (int idx = threadIdx.x; idx < kNB * kNB / 2; idx += kCholThreads) {
            const int r = idx >> 5, c = (idx & 31) * 2;
            const bool ok = r0 + r < n && c0 + c < n;      // n is even on this path: a pair never straddles n
            cp_async16_cg(dst + r * kCholLd + c, ok ? A + (int64_t)(r0 + r) * ld + c0 + c : A, ok);
        }
    } else {
        for (int idx = threadIdx.x; idx < kNB * kNB; idx += kCholThreads) {
            const int r = idx >> 6, c = idx & 63;
            const bool ok = r0 + r < n && c0 + c < n;
            cp_async8(dst + r * kCholLd + c, ok ? A + (int64_t)(r0 + r) * ld + c0 + c : A, ok);
        }
    }
}

// Step P of the strip factorisation: row P of the diagonal block is published, every thread scales its own entry
// of that row and eliminates it from the rows below.
template <int P>
__device__ __forceinline__ void chol_strip_step(double (&col)[kNB], double* rowbuf, bool is_diag, int tid, int g,
                                                int k0, int32_t* status) {
    double* rb = rowbuf + (P & 1) * kNB;
    if (is_diag) rb[tid] = col[P];
    __syncthreads();
    double d = rb[P];
    if (!(d > 0.0) || !isfinite(d)) {
        if (tid == 0 && g == 0) report(status, PTQ_ERR_NOT_SPD, k0 + P);
        d = 1.0;
    }
    const double inv = 1.0 / d;
    const double t = col[P] * inv;
    col[P] = col[P] * sqrt(inv);                                  // U[P][c]
#pragma unroll
    for (int i = P + 1; i < kNB; ++i) col[i] = fma(-rb[i], t, col[i]);
}
template <int... Ps>
__device__ __forceinline__ void chol_strip_steps(double (&col)[kNB], double* rowbuf, bool is_diag, int tid, int g,
                                                 int k0, int32_t* status, std::integer_sequence<int, Ps...>) {
    (chol_strip_step<Ps>(col, rowbuf, is_diag, tid, g, k0, status), ...);
}

__global__ void __launch_bounds__(kCholThreads, 1)
chol_coop_kernel(double* __restrict__ A, int n, int64_t ld, int vec16, unsigned* bar, int32_t* status) {
    extern __shared__ __align__(16) unsigned char chol_smem_raw[];
    double* opnd = reinterpret_cast<double*>(chol_smem_raw);                // [2 stages][2 operands][64][kCholLd]
    double* rowbuf = opnd + 2 * 2 * kNB * kCholLd;                          // [2][64]
    int* s_flag = reinterpret_cast<int*>(rowbuf + 2 * kNB);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = gridDim.x;
    const int nb = (n + kNB - 1) / kNB;
    unsigned epoch = 0;

    for (int k = 0; k < nb; ++k) {
        const int k0 = k * kNB;
        // ------------------------------------------------------------------ strip phase
        const int panel_cols = n - k0 - kNB;                                // columns to the right of the block
        const int groups = panel_cols > 0 ? (panel_cols + kCholPanelCols - 1) / kCholPanelCols : 0;
        const int reps = groups > 0 ? groups : 1;                            // last block: diagonal only
        for (int g = blockIdx.x; g < reps; g += G) {
            // column owned by this thread: tid < 64 -> diagonal block column tid, else a panel column
            const bool is_diag = tid < kNB;
            const int gc = is_diag ? k0 + tid : k0 + kNB + g * kCholPanelCols + (tid - kNB);
            const bool live = gc < n && (is_diag || groups > 0);
            double col[kNB];
#pragma unroll
            for (int p = 0; p < kNB; ++p) {
                double v = (is_diag && p == tid) ? 1.0 : 0.0;                // identity padding below n
                if (live && k0 + p < n && (!is_diag || p <= tid)) v = __ldcg(A + (int64_t)(k0 + p) * ld + gc);
                col[p] = v;
            }
            chol_strip_steps(col, rowbuf, is_diag, tid, g, k0, status, std::make_integer_sequence<int, kNB>());
            if (live) {
                if (is_diag) {
                    if (g == 0) {
#pragma unroll
                        for (int p = 0; p < kNB; ++p)
                            if (p <= tid && k0 + p < n) __stcg(A + (int64_t)(k0 + p) * ld + gc, col[p]);
                    }
                } else {
#pragma unroll
                    for (int p = 0; p < kNB; ++p)
                        if (k0 + p < n) __stcg(A + (int64_t)(k0 + p) * ld + gc, col[p]);
                }
            }
            __syncthreads();     // rowbuf is reused by the next repetition
        }
        if (k == nb - 1) break;
        ++epoch;
        if (!grid_barrier(bar, epoch * (unsigned)G, s_flag)) break;

        // ------------------------------------------------------------------ trailing phase
        const int m = nb - 1 - k;
        const int T = m * (m + 1) / 2;
        auto tile_ij = [&](int t, int& bi, int& bj) {
            int i = k + 1, rem = t;
            while (rem >= nb - i) { rem -= nb - i; ++i; }
            bi = i; bj = i + rem;
        };
        int stage = 0;
        if ((int)blockIdx.x < T) {
            int bi, bj;
            tile_ij(blockIdx.x, bi, bj);
            chol_load_block(opnd, A, ld, n, k0, bi * kNB, vec16);
            chol_load_block(opnd + kNB * kCholLd, A, ld, n, k0, bj * kNB, vec16);
        }
        cp_async_commit();
        for (int t = blockIdx.x; t < T; t += G) {
            int bi, bj;
            tile_ij(t, bi, bj);
            if (t + G < T) {
                int ni, nj;
                tile_ij(t + G, ni, nj);
                double* nxt = opnd + (stage ^ 1) * 2 * kNB * kCholLd;
                chol_load_block(nxt, A, ld, n, k0, ni * kNB, vec16);
                chol_load_block(nxt + kNB * kCholLd, A, ld, n, k0, nj * kNB, vec16);
            }
            cp_async_commit();
            cp_async_wait<1>();
            __syncthreads();
            const double* as = opnd + stage * 2 * kNB * kCholLd;            // as[kk][m] = U[k0 + kk][i0 + m]
            const double* bs = as + kNB * kCholLd;                           // bs[kk][n] = U[k0 + kk][j0 + n]
            const int wm0 = (warp >> 2) * 32, wn0 = (warp & 3) * 16;
            const int lq = lane >> 2, lr = lane & 3;
            double acc[4][2][2];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 2; ++b) acc[a][b][0] = acc[a][b][1] = 0.0;
#pragma unroll 4
            for (int kk = 0; kk < kNB; kk += 4) {
                double af[4], bf[2];
#pragma unroll
                for (int a = 0; a < 4; ++a) af[a] = as[(kk + lr) * kCholLd + wm0 + a * 8 + lq];
#pragma unroll
                for (int b = 0; b < 2; ++b) bf[b] = bs[(kk + lr) * kCholLd + wn0 + b * 8 + lq];
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 2; ++b) dmma_884(acc[a][b][0], acc[a][b][1], af[a], bf[b]);
            }
            const int i0 = bi * kNB, j0 = bj * kNB;
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int r = wm0 + a * 8 + lq;
#pragma unroll
                for (int b = 0; b < 2; ++b)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int c = wn0 + b * 8 + 2 * lr + e;
                        if (i0 + r < n && j0 + c < n && (bi != bj || c >= r)) {
                            double* dst = A + (int64_t)(i0 + r) * ld + j0 + c;
                            __stcg(dst, __ldcg(dst) - acc[a][b][e]);
                        }
                    }
            }
            __syncthreads();     // all warps are done with this stage before it is refilled
            stage ^= 1;
        }
        cp_async_wait<0>();
        ++epoch;
        if (!grid_barrier(bar, epoch * (unsigned)G, s_flag)) break;
    }
    cp_async_wait<0>();
    if (tid == 0 && ld_acquire_u32(&bar[1]) != 0u) report(status, PTQ_ERR_TIMEOUT, blockIdx.x, 1);
}

// In-place blocked upper Cholesky of the n x n matrix A (row stride n).  Only the upper triangle is read or
// written.  `bar` is 2 x uint32 of device scratch.
inline int cholesky_upper(double* A, int n, unsigned* bar, int32_t* status, cudaStream_t stream) {
    static int grid = 0;
    if (grid == 0) {
        if (cudaFuncSetAttribute(chol_coop_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kCholSmemBytes) != cudaSuccess)
            return PTQ_ERR_CUDA;
        int dev = 0, sms = 0, per_sm = 0, coop = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
        if (!coop) return PTQ_ERR_UNSUPPORTED;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, chol_coop_kernel, kCholThreads, kCholSmemBytes) !=
                cudaSuccess || per_sm < 1)
            return PTQ_ERR_CUDA;
        grid = sms;          // one CTA per SM: the cooperative launch guarantees that all of them are resident
    }
    if (cudaMemsetAsync(bar, 0, 2 * sizeof(unsigned), stream) != cudaSuccess) return PTQ_ERR_CUDA;
    int64_t ld = n;
    int vec16 = ((n & 1) == 0 && aligned16(A)) ? 1 : 0;
    void* args[] = {&A, &n, &ld, &vec16, &bar, &status};
    Launch l(K_CHOL_COOP, stream);
    if (cudaLaunchCooperativeKernel((const void*)chol_coop_kernel, dim3(grid), dim3(kCholThreads), args,
                                    kCholSmemBytes, stream) != cudaSuccess) {
        cudaGetLastError();
        return PTQ_ERR_CUDA;
    }
    return PTQ_OK;
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
