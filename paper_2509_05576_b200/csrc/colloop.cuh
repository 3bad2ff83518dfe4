// The column-synchronous quantization sweep (Sec. 4.2 steps 3-5, Eq. 11 / Eq. 12) in blocked form.
//
// With A the permuted inverse Hessian and A = U^T U its upper Cholesky factor, the matrix that Eq. 12 leaves
// before step p has row p equal to sqrt(pivot) * U[p, p:], so Eq. 11 for column p reads
//     e_i = (w_ip - q_ip) / U[p][p],      w_ij -= e_i * U[p][j]   for j > p.
// Columns are processed in blocks of 64; the effect of a block on a later block is one float64 MMA tile,
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

// A[a][b] = Hinv[perm[a]][perm[b]] for b from the start of row a's 64-column diagonal tile on: the factorisation and
// everything after it read the upper triangle only (whole 64 x 64 tiles on the diagonal), the rest of A is left alone.
__global__ void gather_sym_kernel(const double* __restrict__ Hinv, const int32_t* __restrict__ perm, int n,
                                  double* __restrict__ A) {
    const int a = blockIdx.y;
    const int b_first = a & ~(kNB - 1);
    const int64_t src = (int64_t)clamp_index(perm[a], n) * n;
    for (int b = b_first + blockIdx.x * blockDim.x + threadIdx.x; b < n; b += gridDim.x * blockDim.x)
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
// quantizes it, writes the scaled errors E[:, b] and the codes, eight columns at a time, and raises the group's counter
// with every piece (8 b + 8 once the block is complete).  Every CTA
// of the group then applies E[:, b] to the blocks IT owns: W[:, b'] -= E[:, b] U[b, b'] (the deferred part of Eq. 11),
// a 32 x 64 x 64 float64 tensor-core MMA tile per block.  All updates of one block are made by its owner, in order, so
// no block is ever touched by two CTAs; the only cross-CTA dependency is "E[:, b] is ready".  The owner of block b + 1
// updates that block first, straight into registers, and starts quantizing at once; its other blocks catch up later.
// Waits on the counter are bounded; when one expires the CTA raises the abort word, reports PTQ_ERR_TIMEOUT and leaves.
//
// Inside a block the 32 x 64 tile of W lives in registers as 8 x 8 MMA accumulator fragments, warp k holding columns
// 8 k .. 8 k + 7 of all 32 rows.  Columns are quantized eight at a time ("mini-block" m, owned by warp m):
//   - warp m turns its fragments into one-row-per-lane form and runs the eight dependent steps
//         c = clamp(rint(w / s) + z),  d = w - q,  w_j -= d U[p][j] / U[p][p]   (j inside the mini-block),
//     with warp-private shared-memory staging only, then publishes the 32 x 8 differences d;
//   - the warps to its right subtract d (U[p][j] / U[p][p]) from their fragments: a rank-8 update, two MMAs per
//     fragment.  One barrier per mini-block, among the warps from m rightwards only.
// ------------------------------------------------------------------------------------------------------------
constexpr int kSweepThreads = 256;
constexpr int kSweepRows = 32;
constexpr int kSweepLd = kNB + 4;                                   // 68: conflict-free MMA operand stride
constexpr int kSweepTLd = 9;                                        // fragment <-> row-per-lane staging
constexpr int kSweepDLd = 12;                                       // 32 x 8 differences as MMA operand A
constexpr int kSweepSmemDoubles = kNB * kSweepLd /*Us*/ + kNB /*rdiag*/ +
                                  kSweepRows * kSweepTLd /*T*/ + 2 * kSweepRows * kSweepDLd /*Dm*/ +
                                  kSweepRows * kSweepLd /*Ea*/ + 2 * kNB * kSweepLd /*Bb*/;
constexpr size_t kSweepSmemBytes = sizeof(double) * kSweepSmemDoubles + kSweepRows * (kNB + 4) + 16;

struct SweepParams {
    double* Wp;             // [rows x n] permuted weights, float64, updated in place
    const double* U;        // [n x n] upper Cholesky factor of the permuted inverse Hessian
    double* E;              // [rows x n] scaled errors
    uint8_t* codes_p;       // [rows x n] codes in permuted order
    const float* scale;
    const float* zero;
    int rows, n, bits, vec16;     // n: columns to sweep (the first n of each row)
    int64_t ld;                   // row stride of Wp, U, E and codes_p (>= n)
    unsigned* flags;        // [groups] published 8-column pieces of E per group, then [1] abort word; zero at launch
    int32_t* status;
    long long spin_limit;   // SM clock cycles after which a wait on another CTA gives up
};

// Waits (one thread) until *counter >= target.  Gives up when the abort word is raised or after spin_limit cycles, in
// which case it raises the abort word itself.  Returns whether the target was reached.
__device__ __forceinline__ bool bounded_counter_wait(const unsigned* counter, unsigned target, unsigned* abort_word,
                                                     long long spin_limit) {
    const long long t0 = clock64();
    unsigned it = 0;
    while (ld_acquire_u32(counter) < target) {
        if ((++it & 63u) == 0u) {
            if (ld_acquire_u32(abort_word) != 0u) return false;
            if (clock64() - t0 > spin_limit) { atomicExch(abort_word, 1u); return false; }
        }
    }
    return true;
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

__device__ __forceinline__ double ld_relaxed_f64(const double* p) {
    double v;
    asm volatile("ld.relaxed.gpu.global.f64 %0, [%1];" : "=d"(v) : "l"(p) : "memory");
    return v;
}

// Per-row constants of the quantizer: scale, 1 / scale, zero-point and the clamp range [-z, maxq - z] of rint(w / s)
// (clamping that integer is the same as clamping the code to [0, maxq], because the zero-point is an integer).
struct RowGrid {
    double sc, rsc, zp, lo, hi;
};

// Eight dependent quantization steps of one row (one lane) on the mini-block whose weights are v[0..7].
// us points at U'[8 m][8 m] (rows of U divided by their pivots, row stride kSweepLd).  Returns the differences
// d_p = w_p - q_p in v[] and the clamped level indices in lev[].
//
// EXACT = false: the level index rint(w / s) -- by definition a true float64 division -- is taken from the product
// w * (1 / s), which differs from the quotient by less than 4e-16 |w / s|; whenever the product is further than 1e-6
// from a rounding boundary (and below 1e9 in magnitude) both round to the same integer.  The return value tells whether
// some step was closer than that, in which case the caller repeats the mini-block with EXACT = true (the division).
// Rounding: (v + 1.5 * 2^52) - 1.5 * 2^52 is round-to-nearest-even for |v| < 2^51.
template <bool EXACT>
__device__ __forceinline__ bool sweep_chain8(double (&v)[8], double (&lev)[8], const double* us, const RowGrid& g) {
    bool danger = false;
#pragma unroll
    for (int p = 0; p < 8; ++p) {
        double rv;
        if (EXACT) {
            rv = rint(v[p] / g.sc);
        } else {
            const double t = v[p] * g.rsc;
            rv = (t + 6755399441055744.0) - 6755399441055744.0;
            danger |= !(fabs(t - rv) < 0.5 - 1e-6) || !(fabs(t) < 1e9);
        }
        const double rvc = fmin(fmax(rv, g.lo), g.hi);
        const double d = v[p] - g.sc * rvc;
#pragma unroll
        for (int j = p + 1; j < 8; ++j) v[j] = fma(-d, us[p * kSweepLd + j], v[j]);
        v[p] = d;
        lev[p] = rvc;
    }
    return danger;
}

__global__ void __launch_bounds__(kSweepThreads, 1) sweep_coop_kernel(SweepParams prm) {
    extern __shared__ __align__(16) unsigned char sweep_smem[];
    double* Us = reinterpret_cast<double*>(sweep_smem);                // [64][68] diagonal block of U, rows / pivot
    double* rdiag = Us + kNB * kSweepLd;                               // [64] 1 / U_pp
    double* T = rdiag + kNB;                          // [32][9] staging of the current mini-block
    double* Dm = T + kSweepRows * kSweepTLd;                           // [2][32][12] differences of a mini-block
    double* Ea = Dm + 2 * kSweepRows * kSweepDLd;                      // [32][68] MMA operand A: E[:, e]
    double* Bb = Ea + kSweepRows * kSweepLd;                           // [2][64][68] MMA operand B: U[e, b']
    uint8_t* Cs = reinterpret_cast<uint8_t*>(Bb + 2 * kNB * kSweepLd); // [32][68] codes of the block
    int* s_flag = reinterpret_cast<int*>(Cs + kSweepRows * (kNB + 4));
    volatile int* s_pub = s_flag + 1;                                  // last piece of E this CTA has announced

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rows = prm.rows, n = prm.n;
    const int64_t ld = prm.ld;
    const int nb = (n + kNB - 1) / kNB;
    const int groups = (rows + kSweepRows - 1) / kSweepRows;
    const int G = gridDim.x;
    unsigned* abort_word = prm.flags + groups;
    const double maxq = (double)((1 << prm.bits) - 1);
    const int lq = lane >> 2, lr = lane & 3;
    // far-update MMA tile coordinates: 8 warps as 2 x 4, each 16 x 16
    const int wm0 = (warp >> 2) * 16, wn0 = (warp & 3) * 16;

    int cpg = 1, g_first = blockIdx.x, g_step = G, ci = 0;
    if (groups < G) {
        const int per = G / groups;                // CTAs reserved per group; only the first cpg of them work
        cpg = per < nb ? per : nb;
        g_first = blockIdx.x / per;
        ci = blockIdx.x - g_first * per;
        g_step = groups;                           // one group per CTA
        if (g_first >= groups || ci >= cpg) return;
    }

    // diagonal block of U for block b: Us = rows divided by their pivots, rdiag = 1 / pivot
    auto load_diag = [&](int b) {
        const int p0 = b * kNB;
        const int kb = n - p0 < kNB ? n - p0 : kNB;
        for (int idx = tid; idx < kNB * kNB; idx += kSweepThreads) {
            const int r = idx >> 6, c = idx & 63;
            double v = (r == c) ? 1.0 : 0.0;
            if (r < kb && c < kb && c >= r) v = __ldcg(prm.U + (int64_t)(p0 + r) * ld + p0 + c);
            Us[r * kSweepLd + c] = v;
        }
        __syncthreads();
        if (tid < kNB) rdiag[tid] = 1.0 / Us[tid * kSweepLd + tid];
        __syncthreads();
        for (int idx = tid; idx < kNB * kNB; idx += kSweepThreads) Us[(idx >> 6) * kSweepLd + (idx & 63)] *= rdiag[idx >> 6];
    };

    for (int g = g_first; g < groups; g += g_step) {
        const int r0 = g * kSweepRows;
        // the grid of this lane's row (one row per lane in the chains), fixed for the whole group
        const int row = r0 + lane;
        const bool live = row < rows;
        RowGrid rg;
        rg.sc = live ? (double)prm.scale[row] : 1.0;
        rg.zp = live ? (double)prm.zero[row] : 0.0;
        rg.rsc = 1.0 / rg.sc;
        rg.lo = -rg.zp;
        rg.hi = maxq - rg.zp;
        int lazy = 0;
        bool prepared = false;           // Us / rdiag / blk already hold the block about to be quantized
        bool ahead = false;              // blk holds this CTA's next block with E of the block before last folded in
        // the block being quantized: fragment a = rows 8 a + lq, columns 8 warp + 2 lr + {0, 1}
        double blk[4][2];
        for (int b = 0; b < nb; ++b) {
            const int p0 = b * kNB;
            const int kb = n - p0 < kNB ? n - p0 : kNB;
            const bool mine = (b % cpg) == ci;
            const bool next_mine = cpg > 1 && b + 1 < nb && ((b + 1) % cpg) == ci;
            // With four or more CTAs in the group, the owner of block b + 2 folds E[:, b] into that block while block b
            // is still being quantized, just as the owner of block b + 1 does: the deferred update of a block by the two
            // blocks before it then never waits for the group's counter, which is what used to delay its owner.
            const bool next2_mine = cpg >= 4 && b + 2 < nb && ((b + 2) % cpg) == ci;
            if (next2_mine) {
                __syncthreads();
                sweep_load_tile(Bb, kSweepLd, prm.U, ld, p0, p0 + 2 * kNB, kNB, kNB, n, n, prm.vec16);
                cp_async_commit();
                load_diag(b + 2);            // nothing of it depends on E: out of the way two blocks early
            }
            if (next_mine) {
                // block b + 1 is quantized here next: what does not depend on E[:, b] is fetched before waiting for it
                __syncthreads();
                sweep_load_tile(Bb, kSweepLd, prm.U, ld, p0, p0 + kNB, kNB, kNB, n, n, prm.vec16);
                cp_async_commit();
                if (!ahead) load_diag(b + 1);
            }
            if (mine) {
                // ------------------------------------------------------------ quantize block b
                if (!prepared) {
                    __syncthreads();
                    load_diag(b);
#pragma unroll
                    for (int a = 0; a < 4; ++a)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int r = r0 + 8 * a + lq, c = p0 + 8 * warp + 2 * lr + e;
                            blk[a][e] = (r < rows && c < n) ? __ldcg(prm.Wp + (int64_t)r * ld + c) : 0.0;
                        }
                }
                __syncthreads();
#pragma unroll
                for (int m = 0; m < 8; ++m) {
                    double* dm = Dm + (m & 1) * kSweepRows * kSweepDLd;
                    double v[8];
                    if (warp < m) continue;          // this warp's columns are done; it is out of the remaining barriers
                    if (warp == m) {
                        // fragments -> one row per lane
#pragma unroll
                        for (int a = 0; a < 4; ++a)
#pragma unroll
                            for (int e = 0; e < 2; ++e) T[(8 * a + lq) * kSweepTLd + 2 * lr + e] = blk[a][e];
                        __syncwarp();
                        double lev[8];
#pragma unroll
                        for (int c = 0; c < 8; ++c) v[c] = T[lane * kSweepTLd + c];
                        const double* us = Us + (8 * m) * kSweepLd + 8 * m;
                        const bool danger = sweep_chain8<false>(v, lev, us, rg);
                        if (__any_sync(0xffffffffu, danger)) {
#pragma unroll
                            for (int c = 0; c < 8; ++c) v[c] = T[lane * kSweepTLd + c];
                            sweep_chain8<true>(v, lev, us, rg);
                        }
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            dm[lane * kSweepDLd + c] = v[c];
                            Cs[lane * (kNB + 4) + 8 * m + c] = (uint8_t)(int)(lev[c] + rg.zp);
                        }
                    }
                    // the differences of mini-block m become visible to the warps right of it (only those take part)
                    if (m < 7) asm volatile("bar.sync 1, %0;" ::"r"((8 - m) * 32) : "memory");
                    if (warp == m) {
                        // The scaled errors e = d / U_pp of these eight columns go out at once, off the critical path
                        // (the warps to the right are already updating): the owner of the next block folds them into its
                        // block while the rest of this block is still being quantized.
                        if (live) {
                            double* dst = prm.E + (int64_t)row * ld + p0 + 8 * m;
#pragma unroll
                            for (int c = 0; c < 8; ++c) {
                                v[c] *= rdiag[8 * m + c];
                                v[c] = v[c] == v[c] ? v[c] : 0.0;        // E starts out as NaN = "not there yet"
                            }
                            if (prm.vec16 && p0 + 8 * m + 8 <= n) {
#pragma unroll
                                for (int c = 0; c < 8; c += 2)
                                    __stcg(reinterpret_cast<double2*>(dst + c), make_double2(v[c], v[c + 1]));
                            } else {
#pragma unroll
                                for (int c = 0; c < 8; ++c)
                                    if (p0 + 8 * m + c < n) __stcg(dst + c, v[c]);
                            }
                        }
                        if (cpg > 1) {
                            __threadfence();
                            __syncwarp();
                            if (lane == 0) {
                                // The counter must rise in order: piece m leaves only after piece m - 1 of this block
                                // (whose fence may have taken longer than this warp's whole chain), else a reader
                                // could be told of columns that are not visible yet, or see the counter fall back.
                                if (m > 0) {
                                    const long long t0 = clock64();
                                    while (*s_pub != 8 * b + m) {
                                        if (clock64() - t0 > prm.spin_limit) { atomicExch(abort_word, 1u); break; }
                                    }
                                }
                                // a reduction without a return value: the warp does not wait for the round trip, and
                                // should two of them overtake each other on the way the maximum is still right (the
                                // data of the earlier piece was fenced before its warp let this one pass)
                                atomicMax(&prm.flags[g], (unsigned)(8 * b + m + 1));
                                *s_pub = 8 * b + m + 1;
                            }
                        }
                    } else {
                        // rank-8 update of this warp's columns: blk -= d (U'[8 m .. 8 m + 7][8 warp .. 8 warp + 7])
                        const double b0 = Us[(8 * m + lr) * kSweepLd + 8 * warp + lq];
                        const double b1 = Us[(8 * m + 4 + lr) * kSweepLd + 8 * warp + lq];
#pragma unroll
                        for (int a = 0; a < 4; ++a) {
                            const double a0 = -dm[(8 * a + lq) * kSweepDLd + lr];
                            const double a1 = -dm[(8 * a + lq) * kSweepDLd + 4 + lr];
                            dmma_884(blk[a][0], blk[a][1], a0, b0);
                            dmma_884(blk[a][0], blk[a][1], a1, b1);
                        }
                    }
                }
                __syncthreads();
                for (int idx = tid; idx < kSweepRows * kNB; idx += kSweepThreads) {
                    const int r = idx >> 6, c = idx & 63;
                    if (r0 + r < rows && c < kb) prm.codes_p[(int64_t)(r0 + r) * ld + p0 + c] = Cs[r * (kNB + 4) + c];
                }
                prepared = false;
            } else if (!next_mine && !next2_mine) {
                // ------------------------------------------------------------ wait for all of E[:, b]
                if (tid == 0) {
                    const int ok = bounded_counter_wait(&prm.flags[g], (unsigned)(8 * (b + 1)), abort_word,
                                                        prm.spin_limit) ? 1 : 0;
                    __threadfence();
                    *s_flag = ok;
                }
                __syncthreads();
                if (*s_flag == 0) {
                    cp_async_wait<0>();
                    if (tid == 0) report(prm.status, PTQ_ERR_TIMEOUT, blockIdx.x, 2);
                    return;
                }
            }
            if (b + 1 >= nb) break;
            // ---------------------------------------------------------------- deferred Eq. 11 on the owned blocks
            if (next_mine || next2_mine) {
                // block b + 1 (or b + 2) only, straight into the fragments the chain starts from; the other blocks catch
                // up later
                if (!(next_mine && ahead)) {
                    const int c0 = p0 + (next_mine ? kNB : 2 * kNB);
#pragma unroll
                    for (int a = 0; a < 4; ++a)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int r = r0 + 8 * a + lq, c = c0 + 8 * warp + 2 * lr + e;
                            blk[a][e] = (r < rows && c < n) ? __ldcg(prm.Wp + (int64_t)r * ld + c) : 0.0;
                        }
                }
                // whatever of E[:, b] is out already comes in one go through shared memory (an owner that arrives late
                // would otherwise pay one L2 round trip per piece); the pieces still missing there are polled below
                sweep_load_tile(Ea, kSweepLd, prm.E, ld, r0, p0, kSweepRows, kNB, rows, n, prm.vec16);
                cp_async_commit();
                cp_async_wait<0>();
                __syncthreads();             // U[b, b + 1] (or U[b, b + 2]) is in Bb, the snapshot of E[:, b] in Ea
                // E[:, b] arrives eight columns at a time.  Every warp polls the group's counter for itself (bounded),
                // requests the operand of piece m straight from global memory as soon as it is out, and meanwhile
                // multiplies piece m - 1, whose operand was requested one piece earlier.
                double prod[4][2], af[2][2][4];        // af[piece parity][k step][row fragment]
#pragma unroll
                for (int a = 0; a < 4; ++a) prod[a][0] = prod[a][1] = 0.0;
                bool ok = true;
#pragma unroll
                for (int m = 0; m <= 8; ++m) {
                    if (m < 8) {
                        // E is NaN until written: the operand of piece m is read again and again until none of this
                        // warp's values is NaN any more, which needs neither the publisher's fence nor its counter
                        // (those serve the CTAs that pick E up later, off the critical path).  Bounded.
                        bool snap = true;
#pragma unroll
                        for (int s4 = 0; s4 < 2; ++s4)
#pragma unroll
                            for (int a = 0; a < 4; ++a) {
                                const double x = Ea[(8 * a + lq) * kSweepLd + 8 * m + 4 * s4 + lr];
                                af[m & 1][s4][a] = x;
                                snap = snap && x == x;
                            }
                        const long long t0 = clock64();
                        unsigned it = 0;
                        while (!__all_sync(0xffffffffu, snap)) {
                            bool have = true;
#pragma unroll
                            for (int s4 = 0; s4 < 2; ++s4)
#pragma unroll
                                for (int a = 0; a < 4; ++a) {
                                    const int r = r0 + 8 * a + lq;
                                    const double x =
                                        r < rows ? ld_relaxed_f64(prm.E + (int64_t)r * ld + p0 + 8 * m + 4 * s4 + lr) : 0.0;
                                    af[m & 1][s4][a] = x;
                                    have = have && x == x;
                                }
                            if (__all_sync(0xffffffffu, have)) break;
                            if ((++it & 15u) == 0u) {
                                bool bad = ld_acquire_u32(abort_word) != 0u;
                                if (!bad && clock64() - t0 > prm.spin_limit) { atomicExch(abort_word, 1u); bad = true; }
                                if (__any_sync(0xffffffffu, bad)) { ok = false; break; }
                            }
                        }
                        if (!ok) break;
                    }
                    if (m > 0) {
#pragma unroll
                        for (int s4 = 0; s4 < 2; ++s4) {
                            const double bf = Bb[(8 * (m - 1) + 4 * s4 + lr) * kSweepLd + 8 * warp + lq];
#pragma unroll
                            for (int a = 0; a < 4; ++a) dmma_884(prod[a][0], prod[a][1], af[(m - 1) & 1][s4][a], bf);
                        }
                    }
                }
                if (__syncthreads_or(ok ? 0 : 1)) {
                    if (tid == 0) report(prm.status, PTQ_ERR_TIMEOUT, blockIdx.x, 3);
                    return;
                }
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    blk[a][0] -= prod[a][0];
                    blk[a][1] -= prod[a][1];
                }
                prepared = next_mine;
                ahead = !next_mine;
                continue;
            }
            const int b_first = b + 1 + (((ci - (b + 1)) % cpg) + cpg) % cpg;     // first owned block beyond b
            if (b_first >= nb) break;                                               // nothing left for this CTA
            const int e_lo = lazy;
            lazy = b + 1;
            for (int e = e_lo; e <= b; ++e) {
                // operand A: E[r0 .. r0+31][64 e .. 64 e + 63]
                __syncthreads();
                sweep_load_tile(Ea, kSweepLd, prm.E, ld, r0, e * kNB, kSweepRows, kNB, rows, n, prm.vec16);
                int stage = 0;
                sweep_load_tile(Bb, kSweepLd, prm.U, ld, e * kNB, b_first * kNB, kNB, kNB, n, n, prm.vec16);
                cp_async_commit();
                for (int bp = b_first; bp < nb; bp += cpg) {
                    if (bp + cpg < nb)
                        sweep_load_tile(Bb + (stage ^ 1) * kNB * kSweepLd, kSweepLd, prm.U, ld, e * kNB,
                                        (bp + cpg) * kNB, kNB, kNB, n, n, prm.vec16);
                    cp_async_commit();
                    // old values of the tile first (their latency hides behind the MMAs)
                    const int j0 = bp * kNB;
                    double old[2][2][2], acc[2][2][2];
                    bool keep[2][2][2];
#pragma unroll
                    for (int a = 0; a < 2; ++a) {
                        const int r = r0 + wm0 + a * 8 + lq;
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const int c = j0 + wn0 + q * 8 + 2 * lr;
                            keep[a][q][0] = r < rows && c < n;
                            keep[a][q][1] = r < rows && c + 1 < n;
                            const double* src = prm.Wp + (int64_t)r * ld + c;
                            if (prm.vec16 && keep[a][q][0]) {
                                const double2 v = __ldcg(reinterpret_cast<const double2*>(src));
                                old[a][q][0] = v.x;
                                old[a][q][1] = v.y;
                            } else {
                                old[a][q][0] = keep[a][q][0] ? __ldcg(src) : 0.0;
                                old[a][q][1] = keep[a][q][1] ? __ldcg(src + 1) : 0.0;
                            }
                            acc[a][q][0] = acc[a][q][1] = 0.0;
                        }
                    }
                    cp_async_wait<1>();
                    __syncthreads();
                    const double* bs = Bb + stage * kNB * kSweepLd;
#pragma unroll 4
                    for (int kk = 0; kk < kNB; kk += 4) {
                        double af[2], bf[2];
#pragma unroll
                        for (int a = 0; a < 2; ++a) af[a] = Ea[(wm0 + a * 8 + lq) * kSweepLd + kk + lr];
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
                            double* dst = prm.Wp + (int64_t)r * ld + c;
                            const double v0 = old[a][q][0] - acc[a][q][0], v1 = old[a][q][1] - acc[a][q][1];
                            if (prm.vec16 && keep[a][q][0]) {
                                __stcg(reinterpret_cast<double2*>(dst), make_double2(v0, v1));
                            } else {
                                if (keep[a][q][0]) __stcg(dst, v0);
                                if (keep[a][q][1]) __stcg(dst + 1, v1);
                            }
                        }
                    }
                    __syncthreads();     // all warps are done with this stage before it is refilled
                    stage ^= 1;
                }
                cp_async_wait<0>();
            }
            __syncthreads();             // the updated blocks are read back through global memory later
        }
    }
}

// Launches the sweep: one CTA per SM, cooperative so that every CTA a waiting CTA depends on is resident.
// n columns are swept; ld (0: n) is the row stride of Wp, U, E and codes_p, so that the first n columns of wider
// arrays can be swept (the rows of U beyond column n are then applied by the caller).
inline int sweep_launch(double* Wp, const double* U, double* E, uint8_t* codes_p, const float* scale, const float* zero,
                        int rows, int n, int bits, unsigned* flags, int32_t* status, cudaStream_t stream,
                        int64_t ld = 0) {
    if (ld == 0) ld = n;
    DeviceState* dev = nullptr;
    int st = current_device_state(&dev);
    if (st) return st;
    if (!dev->coop) return PTQ_ERR_UNSUPPORTED;
    st = ensure_smem_attr(dev, SA_SWEEP, [] {
        cudaError_t e = cudaFuncSetAttribute(sweep_coop_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kSweepSmemBytes);
        int per_sm = 0;
        if (e == cudaSuccess)
            e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sweep_coop_kernel, kSweepThreads, kSweepSmemBytes);
        return (e == cudaSuccess && per_sm < 1) ? cudaErrorLaunchOutOfResources : e;
    });
    if (st) return st;
    // one CTA per SM; with few row groups only the CTAs that get a share of the blocks are launched
    const int groups_l = cdiv(rows, kSweepRows), nb_l = cdiv(n, kNB);
    int grid = coop_cta_budget(dev);
    if (groups_l < grid) {
        const int per = grid / groups_l < nb_l ? grid / groups_l : nb_l;
        grid = groups_l * per;
    }
    const int groups = cdiv(rows, kSweepRows);
    if (cudaMemsetAsync(flags, 0, ((size_t)groups + 1) * sizeof(unsigned), stream) != cudaSuccess) return PTQ_ERR_CUDA;
    // every byte 0xFF is a NaN: "not published yet" for the owner of the next block, which polls the values themselves
    if (cudaMemset2DAsync(E, (size_t)ld * sizeof(double), 0xFF, (size_t)n * sizeof(double), (size_t)rows, stream) !=
        cudaSuccess)
        return PTQ_ERR_CUDA;
    SweepParams prm;
    prm.Wp = Wp; prm.U = U; prm.E = E; prm.codes_p = codes_p; prm.scale = scale; prm.zero = zero;
    prm.rows = rows; prm.n = n; prm.bits = bits; prm.ld = ld;
    prm.vec16 = ((n & 1) == 0 && (ld & 1) == 0 && aligned16(Wp) && aligned16(U) && aligned16(E)) ? 1 : 0;
    prm.flags = flags; prm.status = status; prm.spin_limit = kSpinLimitCycles;
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
