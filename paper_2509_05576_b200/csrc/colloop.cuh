// The column-synchronous quantization sweep (Sec. 4.2 steps 3-5, Eq. 11 / Eq. 12) in blocked form.
//
// With A the permuted inverse Hessian and A = U^T U its upper Cholesky factor, the matrix that Eq. 12 leaves
// before step p has row p equal to sqrt(pivot) * U[p, p:], so Eq. 11 for column p reads
//     e_i = (w_ip - q_ip) / U[p][p],      w_ij -= e_i * U[p][j]   for j > p.
// Columns are processed in blocks of 64: inside a block every row is swept by one thread that keeps the
// block's 64 weights in registers; the effect of the block on a later block is one float64 MMA tile,
// W[:, later] -= E[:, block] U[block, later].
#pragma once
#include "common.cuh"
#include "dgemm.cuh"
#include "order.cuh"
#include "chol.cuh"
#include <utility>

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

// ------------------------------------------------------------------------------------------------------------
// The sweep as ONE persistent cooperative kernel.
//
// Rows never interact (Sec. 4.2 step 4: every row of the current column is quantized at once, independently), so
// the rows are cut into groups of 32 and each group is an independent pipeline.  A group is served by `cpg` CTAs;
// the 64-column blocks are dealt to them round-robin (CTA i owns blocks i, i + cpg, ...).  The owner of block b
//   - quantizes it: one warp, one row per lane, the block's 64 weights in float64 registers, the 64 x 64 diagonal
//     block of U in shared memory: c = clamp(rint(w / s) + z), e = (w - q) / U_pp, w_j -= e U_pj (Eq. 11 inside the
//     block), and writes the scaled errors E[:, b] and the codes;
//   - raises the group's counter to b + 1.
// Every CTA of the group then applies E[:, b] to the blocks IT owns: W[:, b'] -= E[:, b] U[b, b'] (the deferred part
// of Eq. 11), a 32 x 64 x 64 float64 tensor-core MMA tile per block.  All updates of one block are made by its owner,
// in order, so no block is ever touched by two CTAs; the only cross-CTA dependency is "E[:, b] is ready".  The owner of
// block b + 1 updates that block first and starts quantizing at once; its other blocks catch up afterwards.
// Waits on the counter are bounded; when one expires the CTA raises the abort word, reports PTQ_ERR_TIMEOUT and leaves.
// ------------------------------------------------------------------------------------------------------------
constexpr int kSweepThreads = 256;
constexpr int kSweepRows = 32;
constexpr int kSweepLd = kNB + 4;                                   // 68: conflict-free MMA operand stride
constexpr int kSweepWsLd = kNB + 1;                                 // 65: conflict-free row-per-lane access
constexpr size_t kSweepSmemBytes =
    sizeof(double) * (kNB * kNB + kSweepRows * kSweepWsLd + kNB + kSweepRows * kSweepLd + 2 * kNB * kSweepLd) +
    kSweepRows * (kNB + 4) + 16;

struct SweepParams {
    double* Wp;             // [rows x n] permuted weights, float64, updated in place
    const double* U;        // [n x n] upper Cholesky factor of the permuted inverse Hessian
    double* E;              // [rows x n] scaled errors
    uint8_t* codes_p;       // [rows x n] codes in permuted order
    const float* scale;
    const float* zero;
    int rows, n, bits, vec16;
    unsigned* flags;        // [groups] finished blocks per group, then [1] abort word; zero at launch
    int32_t* status;
};

// quant(): the nearest level of the row's grid (ties to even) of w, clamped to the code range.  w / s is a true
// float64 division by definition; the product w * (1 / s) differs from it by less than 4e-16 |w / s|, so whenever that
// product is further than 1e-6 from a rounding boundary (and below 1e9 in magnitude) both round to the same integer and
// the division is skipped.
__device__ __forceinline__ double quant_code_fast(double w, double sc, double rsc, double zp, double maxq) {
    double v = w * rsc;
    double rv = rint(v);
    if (!(fabs(v - rv) < 0.5 - 1e-6) || !(fabs(v) < 1e9)) rv = rint(w / sc);
    double c = rv + zp;
    c = fmax(c, 0.0);
    c = fmin(c, maxq);
    return c;
}

// Copies a tile of nr x nc doubles (nc even when vec16) from src (row stride ld) into dst (row stride dst_ld);
// rows at or beyond rmax and columns at or beyond cmax are filled with zeros.
__device__ __forceinline__ void sweep_load_tile(double* dst, int dst_ld, const double* __restrict__ src, int64_t ld,
                                                int r0, int c0, int nr, int nc, int rmax, int cmax, int vec16) {
    if (vec16) {
        const int half = nc >> 1;
        for (int idx = threadIdx.x; idx < nr * half; idx += kSweepThreads) {
            const int r = idx / half, c = (idx - r * half) * 2;
            const bool ok = r0 + r < rmax && c0 + c < cmax;
            cp_async16_cg(dst + r * dst_ld + c, ok ? src + (int64_t)(r0 + r) * ld + c0 + c : src, ok);
        }
    } else {
        for (int idx = threadIdx.x; idx < nr * nc; idx += kSweepThreads) {
            const int r = idx / nc, c = idx - r * nc;
            const bool ok = r0 + r < rmax && c0 + c < cmax;
            cp_async8(dst + r * dst_ld + c, ok ? src + (int64_t)(r0 + r) * ld + c0 + c : src, ok);
        }
    }
}

template <int... Ps>
__device__ __forceinline__ void sweep_chain_steps(double (&w)[kNB], const double* Us, const double* rdiag, double* ws_row,
                                                  uint8_t* cs_row, double sc, double rsc, double zp, double maxq,
                                                  std::integer_sequence<int, Ps...>) {
    auto step = [&](auto pc) {
        constexpr int P = decltype(pc)::value;
        const double c = quant_code_fast(w[P], sc, rsc, zp, maxq);
        const double q = sc * (c - zp);
        const double e = (w[P] - q) * rdiag[P];
#pragma unroll
        for (int j = P + 1; j < kNB; ++j) w[j] = fma(-e, Us[P * kNB + j], w[j]);
        ws_row[P] = e;
        cs_row[P] = (uint8_t)(int)c;
    };
    (step(std::integral_constant<int, Ps>()), ...);
}

__global__ void __launch_bounds__(kSweepThreads, 1) sweep_coop_kernel(SweepParams prm) {
    extern __shared__ __align__(16) unsigned char sweep_smem[];
    double* Us = reinterpret_cast<double*>(sweep_smem);                // [64][64] diagonal block of U
    double* Ws = Us + kNB * kNB;                                       // [32][65] block of W, later of E
    double* rdiag = Ws + kSweepRows * kSweepWsLd;                      // [64]
    double* Ea = rdiag + kNB;                                          // [32][68] MMA operand A: E[:, e]
    double* Bb = Ea + kSweepRows * kSweepLd;                           // [2][64][68] MMA operand B: U[e, b']
    uint8_t* Cs = reinterpret_cast<uint8_t*>(Bb + 2 * kNB * kSweepLd); // [32][68] codes of the block
    int* s_flag = reinterpret_cast<int*>(Cs + kSweepRows * (kNB + 4));

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rows = prm.rows, n = prm.n;
    const int nb = (n + kNB - 1) / kNB;
    const int groups = (rows + kSweepRows - 1) / kSweepRows;
    const int G = gridDim.x;
    unsigned* abort_word = prm.flags + groups;
    const double maxq = (double)((1 << prm.bits) - 1);

    int cpg = 1, g_first = blockIdx.x, g_step = G, ci = 0;
    if (groups < G) {
        cpg = G / groups;
        if (cpg > nb) cpg = nb;
        const int per = G / groups;                // CTAs reserved per group; only the first cpg of them work
        g_first = blockIdx.x / per;
        ci = blockIdx.x - g_first * per;
        g_step = groups;                           // one group per CTA
        if (g_first >= groups || ci >= cpg) return;
    }

    for (int g = g_first; g < groups; g += g_step) {
        const int r0 = g * kSweepRows;
        int lazy = 0;
        for (int b = 0; b < nb; ++b) {
            const int p0 = b * kNB;
            const int kb = n - p0 < kNB ? n - p0 : kNB;
            const bool mine = (b % cpg) == ci;
            if (mine) {
                // ------------------------------------------------------------ quantize block b
                for (int idx = tid; idx < kNB * kNB; idx += kSweepThreads) {
                    const int r = idx >> 6, c = idx & 63;
                    double v = (r == c) ? 1.0 : 0.0;
                    if (r < kb && c < kb && c >= r) v = __ldcg(prm.U + (int64_t)(p0 + r) * n + p0 + c);
                    Us[idx] = v;
                }
                for (int idx = tid; idx < kSweepRows * kNB; idx += kSweepThreads) {
                    const int r = idx >> 6, c = idx & 63;
                    double v = 0.0;
                    if (r0 + r < rows && c < kb) v = __ldcg(prm.Wp + (int64_t)(r0 + r) * n + p0 + c);
                    Ws[r * kSweepWsLd + c] = v;
                }
                __syncthreads();
                if (tid < kNB) rdiag[tid] = 1.0 / Us[tid * kNB + tid];
                __syncthreads();
                if (warp == 0) {
                    const int row = r0 + lane;
                    const bool live = row < rows;
                    const double sc = live ? (double)prm.scale[row] : 1.0;
                    const double zp = live ? (double)prm.zero[row] : 0.0;
                    const double rsc = 1.0 / sc;
                    double w[kNB];
#pragma unroll
                    for (int c = 0; c < kNB; ++c) w[c] = Ws[lane * kSweepWsLd + c];
                    sweep_chain_steps(w, Us, rdiag, Ws + lane * kSweepWsLd, Cs + lane * (kNB + 4), sc, rsc, zp, maxq,
                                      std::make_integer_sequence<int, kNB>());
                }
                __syncthreads();
                for (int idx = tid; idx < kSweepRows * kNB; idx += kSweepThreads) {
                    const int r = idx >> 6, c = idx & 63;
                    if (r0 + r < rows && c < kb) {
                        __stcg(prm.E + (int64_t)(r0 + r) * n + p0 + c, Ws[r * kSweepWsLd + c]);
                        prm.codes_p[(int64_t)(r0 + r) * n + p0 + c] = Cs[r * (kNB + 4) + c];
                    }
                }
                if (cpg > 1) {
                    __syncthreads();
                    if (tid == 0) {
                        __threadfence();
                        atomicExch(&prm.flags[g], (unsigned)(b + 1));
                    }
                }
            } else {
                // ------------------------------------------------------------ wait for E[:, b]
                if (tid == 0) {
                    const long long t0 = clock64();
                    int ok = 1;
                    unsigned it = 0;
                    while (ld_acquire_u32(&prm.flags[g]) < (unsigned)(b + 1)) {
                        if ((++it & 63u) == 0u) {
                            if (ld_acquire_u32(abort_word) != 0u) { ok = 0; break; }
                            if (clock64() - t0 > 4000000000LL) { atomicExch(abort_word, 1u); ok = 0; break; }
                        }
                    }
                    __threadfence();
                    *s_flag = ok;
                }
                __syncthreads();
                if (*s_flag == 0) {
                    if (tid == 0) report(prm.status, PTQ_ERR_TIMEOUT, blockIdx.x, 2);
                    return;
                }
            }
            if (b + 1 >= nb) break;
            // ---------------------------------------------------------------- deferred Eq. 11 on the owned blocks
            const bool next_mine = cpg > 1 && ((b + 1) % cpg) == ci;
            int e_lo, b_first, b_last;
            if (next_mine) {
                e_lo = b; b_first = b + 1; b_last = b + 1;                 // only the block about to be quantized
            } else {
                e_lo = lazy;
                b_first = b + 1 + (((ci - (b + 1)) % cpg) + cpg) % cpg;     // first owned block beyond b
                b_last = nb - 1;
                lazy = b + 1;
            }
            if (b_first > b_last) {
                // nothing owned beyond b: this CTA is finished with the group once nothing is deferred either
                bool later = false;
                for (int bb = b + 1; bb < nb; ++bb) later |= (bb % cpg) == ci;
                if (!later) break;
                continue;
            }
            for (int e = e_lo; e <= b; ++e) {
                // operand A: E[r0 .. r0+31][64 e .. 64 e + 63]
                __syncthreads();
                sweep_load_tile(Ea, kSweepLd, prm.E, n, r0, e * kNB, kSweepRows, kNB, rows, n, prm.vec16);
                int stage = 0;
                sweep_load_tile(Bb, kSweepLd, prm.U, n, e * kNB, b_first * kNB, kNB, kNB, n, n, prm.vec16);
                cp_async_commit();
                for (int bp = b_first; bp <= b_last; bp += cpg) {
                    if (bp + cpg <= b_last)
                        sweep_load_tile(Bb + (stage ^ 1) * kNB * kSweepLd, kSweepLd, prm.U, n, e * kNB,
                                        (bp + cpg) * kNB, kNB, kNB, n, n, prm.vec16);
                    cp_async_commit();
                    // old values of the tile first (their latency hides behind the MMAs)
                    const int wm0 = (warp >> 2) * 16, wn0 = (warp & 3) * 16;
                    const int lq = lane >> 2, lr = lane & 3;
                    const int j0 = bp * kNB;
                    double acc[2][2][2];
                    bool keep[2][2][2];
#pragma unroll
                    for (int a = 0; a < 2; ++a) {
                        const int r = r0 + wm0 + a * 8 + lq;
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const int c = j0 + wn0 + q * 8 + 2 * lr;
                            keep[a][q][0] = r < rows && c < n;
                            keep[a][q][1] = r < rows && c + 1 < n;
                            const double* src = prm.Wp + (int64_t)r * n + c;
                            if (prm.vec16 && keep[a][q][0]) {
                                const double2 v = __ldcg(reinterpret_cast<const double2*>(src));
                                acc[a][q][0] = v.x;
                                acc[a][q][1] = v.y;
                            } else {
                                acc[a][q][0] = keep[a][q][0] ? __ldcg(src) : 0.0;
                                acc[a][q][1] = keep[a][q][1] ? __ldcg(src + 1) : 0.0;
                            }
                        }
                    }
                    cp_async_wait<1>();
                    __syncthreads();
                    const double* bs = Bb + stage * kNB * kSweepLd;
#pragma unroll 4
                    for (int kk = 0; kk < kNB; kk += 4) {
                        double af[2], bf[2];
#pragma unroll
                        for (int a = 0; a < 2; ++a) af[a] = -Ea[(wm0 + a * 8 + lq) * kSweepLd + kk + lr];
#pragma unroll
                        for (int q = 0; q < 2; ++q) bf[q] = bs[(kk + lr) * kSweepLd + wn0 + q * 8 + lq];
#pragma unroll
                        for (int a = 0; a < 2; ++a)
#pragma unroll
                            for (int q = 0; q < 2; ++q) dmma_884(acc[a][q][0], acc[a][q][1], af[a], bf[q]);
                    }
#pragma unroll
                    for (int a = 0; a < 2; ++a) {
                        const int r = r0 + wm0 + a * 8 + lq;
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const int c = j0 + wn0 + q * 8 + 2 * lr;
                            double* dst = prm.Wp + (int64_t)r * n + c;
                            if (prm.vec16 && keep[a][q][0]) {
                                __stcg(reinterpret_cast<double2*>(dst), make_double2(acc[a][q][0], acc[a][q][1]));
                            } else {
                                if (keep[a][q][0]) __stcg(dst, acc[a][q][0]);
                                if (keep[a][q][1]) __stcg(dst + 1, acc[a][q][1]);
                            }
                        }
                    }
                    __syncthreads();     // all warps are done with this stage before it is refilled
                    stage ^= 1;
                }
                cp_async_wait<0>();
            }
            __syncthreads();             // the updated block is read back through global memory by the next chain
        }
    }
}

// Launches the sweep: one CTA per SM, cooperative so that every CTA a waiting CTA depends on is resident.
inline int sweep_launch(double* Wp, const double* U, double* E, uint8_t* codes_p, const float* scale, const float* zero,
                        int rows, int n, int bits, unsigned* flags, int32_t* status, cudaStream_t stream) {
    static int grid = 0;
    if (grid == 0) {
        if (cudaFuncSetAttribute(sweep_coop_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kSweepSmemBytes) != cudaSuccess)
            return PTQ_ERR_CUDA;
        int dev = 0, sms = 0, per_sm = 0, coop = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
        if (!coop) return PTQ_ERR_UNSUPPORTED;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sweep_coop_kernel, kSweepThreads,
                                                          kSweepSmemBytes) != cudaSuccess || per_sm < 1)
            return PTQ_ERR_CUDA;
        grid = sms;
    }
    const int groups = cdiv(rows, kSweepRows);
    if (cudaMemsetAsync(flags, 0, ((size_t)groups + 1) * sizeof(unsigned), stream) != cudaSuccess) return PTQ_ERR_CUDA;
    SweepParams prm;
    prm.Wp = Wp; prm.U = U; prm.E = E; prm.codes_p = codes_p; prm.scale = scale; prm.zero = zero;
    prm.rows = rows; prm.n = n; prm.bits = bits;
    prm.vec16 = ((n & 1) == 0 && aligned16(Wp) && aligned16(U) && aligned16(E)) ? 1 : 0;
    prm.flags = flags; prm.status = status;
    void* args[] = {&prm};
    Launch l(K_SWEEP_COOP, stream);
    if (cudaLaunchCooperativeKernel((const void*)sweep_coop_kernel, dim3(grid), dim3(kSweepThreads), args,
                                    kSweepSmemBytes, stream) != cudaSuccess) {
        cudaGetLastError();
        return PTQ_ERR_CUDA;
    }
    return PTQ_OK;
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
