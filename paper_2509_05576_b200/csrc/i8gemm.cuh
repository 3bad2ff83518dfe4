// C += alpha * A * B^T for float64 operands on the 5th-generation tensor cores, to float64 accuracy: the deferred part
// of Eq. 11 (W[:, later] -= E[:, block] U[block, later]) and the other large float64 products of the path.
//
// tcgen05 has no float64 kind, so the product is formed the way the Hessian is (gram.cuh): every row a_i of A and
// every row b_j of B is scaled by a power of two 2^sh so that |x| 2^sh < 2^54, rounded to an integer (exact for the
// entries within 2^-54 of the row maximum, an absolute error of at most 2^-55 of the row maximum for the others) and
// written as seven balanced base-256 digits, most significant first.  Then
//     sum_k va_ik vb_jk = sum_{s,t} 256^(12-s-t) (Da_s Db_t^T)_ij ,
// every Da_s Db_t^T is an exact int8 x int8 -> int32 tensor-core product, pairs with s + t = g share one int32 TMEM
// accumulator, groups g <= 6 are kept (28 products; the dropped ones weigh 2^-56 and less), the groups are combined
// exactly in int64, rounded to float64 and scaled by 2^(48 - sh_i - sh_j).  The error of an entry is of the order of
// 2^-54 max|a_i| max|b_j| per term, i.e. that of a float64 dot product; the result is deterministic.
//
// Kernel: one 128 x 64 output tile per CTA iteration.  A TMA producer warp streams 64-wide K blocks of the seven
// slices of both operands (SWIZZLE_64B, 2 stages of 84 KB); one thread issues the 56 tcgen05.mma.kind::i8 of a stage
// into seven TMEM accumulators (7 x 64 columns); four epilogue warps read them back with tcgen05.ld, combine, hand TMEM
// back (the next tile's products then overlap the rest of the epilogue) and add into C through a shared-memory
// transpose, so that the read-modify-write of C is coalesced.  Every mbarrier wait is bounded.
#pragma once
#include "common.cuh"
#include "gram.cuh"

namespace ptq {

constexpr int kXSlices = 7;
constexpr int kXGroups = 7;                  // groups g = s + t = 0..6
constexpr int kXTM = 128, kXTN = 64, kXKB = 64;
constexpr int kXStages = 2;
constexpr int kXABytes = kXTM * kXKB;        // 8 KB per slice
constexpr int kXBBytes = kXTN * kXKB;        // 4 KB per slice
constexpr int kXStageBytes = kXSlices * (kXABytes + kXBBytes);     // 84 KB
constexpr int kXEpiDoubles = 4 * 32 * 17;    // per epilogue warp: 32 rows x 16 columns (+1 padding)
constexpr int kXSmemBytes = kXStages * kXStageBytes + 1024 /*align*/ + 256 /*barriers*/ + kXEpiDoubles * 8;
constexpr int kXThreads = 192;               // warp 0: TMA, warp 1: MMA + TMEM, warps 2..5: epilogue
constexpr int kXShiftTarget = 54;
constexpr int kXMaxK = 16384;                // 7 * 2^14 * 16384 < 2^31

inline size_t i8gemm_plane_bytes(int rows, int k) {
    return (size_t)kXSlices * (size_t)(cdiv(rows, 128) * 128) * (size_t)(cdiv(k, 128) * 128);
}
inline size_t i8gemm_workspace_bytes(int m, int n, int k) {
    return align_up(i8gemm_plane_bytes(m, k)) + align_up(i8gemm_plane_bytes(n, k)) +
           align_up((size_t)(cdiv(m, 128) * 128) * 12) + align_up((size_t)(cdiv(n, 128) * 128) * 12) + 1024;
}
// Output / K-range modes and the slicing of one operand at a time: see XGemmParams, x_slice_operand, x_product below.

__device__ __forceinline__ void x_pack4(const long long (&v)[4], uint32_t (&packed)[kXSlices]) {
#pragma unroll
    for (int s = 0; s < kXSlices; ++s) packed[s] = 0u;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        long long t = v[u];
#pragma unroll
        for (int s = kXSlices - 1; s >= 0; --s) {         // least significant digit first
            const long long d = ((t + 128) & 255) - 128;  // balanced digit in [-128, 127]
            t = (t - d) >> 8;
            packed[s] |= ((uint32_t)(d & 255)) << (8 * u);
        }
    }
}
// Shift of a row whose largest magnitude is m: |x| 2^sh < 2^54 (0 for an all-zero or non-finite row).
__device__ __forceinline__ int x_row_shift(double m) {
    if (!(m > 0.0) || !(m < 1.0e300)) return 0;
    int sh = kXShiftTarget - (ilogb(m) + 1);
    return sh < -900 ? -900 : (sh > 900 ? 900 : sh);
}

// Slices of the rows of X [rows x k] (row stride ld): Q[s][row][kk], one CTA per (padded) row.
__global__ void __launch_bounds__(256) x_slice_rows_kernel(const double* __restrict__ X, int rows, int k, int64_t ld,
                                                            int rows_pad, int k_pad, int8_t* __restrict__ Q,
                                                            int32_t* __restrict__ shifts) {
    __shared__ double smax[256];
    const int row = blockIdx.x;
    const size_t plane = (size_t)rows_pad * k_pad;
    int8_t* q0 = Q + (size_t)row * k_pad;
    if (row >= rows) {
        for (int kk = threadIdx.x * 4; kk < k_pad; kk += 1024)
#pragma unroll
            for (int s = 0; s < kXSlices; ++s) *reinterpret_cast<uint32_t*>(q0 + s * plane + kk) = 0u;
        if (threadIdx.x == 0) shifts[row] = 0;
        return;
    }
    const double* x = X + (int64_t)row * ld;
    double m = 0.0;
    for (int kk = threadIdx.x; kk < k; kk += 256) m = fmax(m, fabs(x[kk]));
    smax[threadIdx.x] = m;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (threadIdx.x < w) smax[threadIdx.x] = fmax(smax[threadIdx.x], smax[threadIdx.x + w]);
        __syncthreads();
    }
    const int sh = x_row_shift(smax[0]);
    const bool dead = sh == 0 && !(smax[0] > 0.0 && smax[0] < 1.0e300);
    if (threadIdx.x == 0) shifts[row] = sh;
    for (int kk = threadIdx.x * 4; kk < k_pad; kk += 1024) {
        long long v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const double xv = (kk + u < k && !dead) ? x[kk + u] : 0.0;
            v[u] = __double2ll_rn(scalbn(xv, sh));
        }
        uint32_t packed[kXSlices];
        x_pack4(v, packed);
#pragma unroll
        for (int s = 0; s < kXSlices; ++s) *reinterpret_cast<uint32_t*>(q0 + s * plane + kk) = packed[s];
    }
}

// Slices of the COLUMNS of X [k x cols] (row stride ld): Q[s][col][kk] -- the operand B of C += A B^T when the matrix
// at hand is stored as [k][j].  Two passes, both over a grid of (32-column groups) x (256-row chunks of k), so that a
// deep operand is spread over many CTAs: x_colmax_kernel takes the column maxima (reads along rows are coalesced; the
// maxima of the chunks meet by an integer atomic maximum on the bit patterns, which orders non-negative doubles as it
// orders integers and does not depend on the order of arrival); x_slice_cols_kernel reads 32 x 32 tiles row-wise, cuts
// them into digits and writes them out transposed through shared memory.
constexpr int kXColChunk = 256;
__global__ void __launch_bounds__(256) x_colmax_kernel(const double* __restrict__ X, int k, int cols, int64_t ld,
                                                        unsigned long long* __restrict__ colmax) {
    __shared__ double smax[8][33];
    const int c0 = blockIdx.x * 32, k0 = blockIdx.y * kXColChunk;
    const int lane = threadIdx.x & 31, wy = threadIdx.x >> 5;
    const int col = c0 + lane;
    const int k1 = k0 + kXColChunk < k ? k0 + kXColChunk : k;
    double m = 0.0;
    if (col < cols)
        for (int kk = k0 + wy; kk < k1; kk += 8) {
            const double a = fabs(X[(int64_t)kk * ld + col]);
            m = a > m || !(a == a) ? a : m;                   // a NaN sticks, so that the column is treated as dead
        }
    smax[wy][lane] = m;
    __syncthreads();
    if (wy == 0 && col < cols) {
        double mm = smax[0][lane];
#pragma unroll
        for (int w = 1; w < 8; ++w) mm = (smax[w][lane] > mm || !(smax[w][lane] == smax[w][lane])) ? smax[w][lane] : mm;
        // NaN and infinity have bit patterns above every finite double: they win the maximum as well
        atomicMax(colmax + col, (unsigned long long)__double_as_longlong(mm));
    }
}
__global__ void __launch_bounds__(256) x_slice_cols_kernel(const double* __restrict__ X, int k, int cols, int64_t ld,
                                                            int cols_pad, int k_pad,
                                                            const unsigned long long* __restrict__ colmax,
                                                            int8_t* __restrict__ Q, int32_t* __restrict__ shifts) {
    __shared__ uint8_t dig[kXSlices][32][36];          // [slice][column][kk within the tile]
    const int c0 = blockIdx.x * 32, kbeg = blockIdx.y * kXColChunk;
    const int lane = threadIdx.x & 31, wy = threadIdx.x >> 5;          // 8 row slices x 32 columns
    const size_t plane = (size_t)cols_pad * k_pad;
    const int col = c0 + lane;
    const double mm = col < cols ? __longlong_as_double((long long)colmax[col]) : 0.0;
    const bool dead = !(mm > 0.0 && mm < 1.0e300);
    const int sh = dead ? 0 : x_row_shift(mm);
    if (blockIdx.y == 0 && wy == 0 && col < cols_pad) shifts[col] = sh;
    const int kend = kbeg + kXColChunk < k_pad ? kbeg + kXColChunk : k_pad;
    for (int k0 = kbeg; k0 < kend; k0 += 32) {
        // thread (wy, lane): rows k0 + wy, + 8, + 16, + 24 of column `col`
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int kk = k0 + wy + 8 * r;
            const double xv = (!dead && kk < k) ? X[(int64_t)kk * ld + col] : 0.0;
            long long t = __double2ll_rn(scalbn(xv, sh));
#pragma unroll
            for (int s = kXSlices - 1; s >= 0; --s) {
                const long long d = ((t + 128) & 255) - 128;
                t = (t - d) >> 8;
                dig[s][lane][wy + 8 * r] = (uint8_t)(d & 255);
            }
        }
        __syncthreads();
        // out: for every slice and column, 32 consecutive bytes; thread -> (column = threadIdx / 8, 4 bytes = threadIdx % 8)
        const int oc = threadIdx.x >> 3, ob = (threadIdx.x & 7) * 4;
        if (c0 + oc < cols_pad) {
#pragma unroll
            for (int s = 0; s < kXSlices; ++s)
                *reinterpret_cast<uint32_t*>(Q + s * plane + (size_t)(c0 + oc) * k_pad + k0 + ob) =
                    *reinterpret_cast<const uint32_t*>(&dig[s][oc][ob]);
        }
        __syncthreads();
    }
}

// Output modes: what the epilogue does with P = A B^T.
enum { X_OUT_ADD_UPPER = 3,  // C += alpha P on the tiles that touch the upper triangle only (A = B, C symmetric, upper kept)
       X_OUT_ADD = 0,        // C += alpha P
       X_OUT_SYM = 1,        // C = alpha P on the tiles that touch the upper triangle, and C[j][i] = C[i][j] (A = B)
       X_OUT_REDUCE = 2 };   // partials[tile] = alpha * sum_ij P_ij D_ij ; C is not touched
// K ranges per tile (operands known to be zero outside them, or terms accounted for elsewhere).
enum { X_K_ALL = 0,
       X_K_FROM_MAX = 1,     // k >= max(i0, j0): A[i][k] = 0 for k < i and B[j][k] = 0 for k < j (a triangular factor)
       X_K_BEFORE_J = 2,     // k < j0: the column blocks before the tile's own
       X_K_OWN_J = 3 };      // j0 <= k < j0 + 64: the tile's own column block
struct XGemmParams {
    double* C;              // [m x n], row stride ldc
    int64_t ldc;
    int m, n, k_pad;
    double alpha;
    const int32_t* sh_a;    // per row of A
    const int32_t* sh_b;    // per row of B
    int32_t* status;
    int out_mode, k_mode;
    const double* D;        // X_OUT_REDUCE: [m x n], row stride ldd
    int64_t ldd;
    double* partials;       // X_OUT_REDUCE: one per tile (0 for tiles without work)
};

// K blocks [kb0, kb1) of tile (bi, bj); an empty range or a tile below the diagonal (X_OUT_SYM) has no work at all.
__device__ __forceinline__ bool x_tile_range(const XGemmParams& prm, int bi, int bj, int nkb, int& kb0, int& kb1) {
    const int i0 = bi * kXTM, j0 = bj * kXTN;
    kb0 = 0;
    kb1 = nkb;
    if ((prm.out_mode == X_OUT_SYM || prm.out_mode == X_OUT_ADD_UPPER) && i0 > j0 + kXTN - 1) return false;
    if (prm.k_mode == X_K_FROM_MAX) kb0 = (i0 > j0 ? i0 : j0) / kXKB;
    else if (prm.k_mode == X_K_BEFORE_J) kb1 = j0 / kXKB;
    else if (prm.k_mode == X_K_OWN_J) { kb0 = j0 / kXKB; kb1 = kb0 + 1; }
    if (kb1 > nkb) kb1 = nkb;
    return kb0 < kb1;
}

__global__ void __launch_bounds__(kXThreads, 1)
i8gemm_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB, XGemmParams prm) {
    extern __shared__ unsigned char xg_smem_raw[];
    const uint32_t raw = smem_u32(xg_smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* base_ptr = xg_smem_raw + (base - raw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + kXStages * kXStageBytes);
    const uint32_t bar0 = base + kXStages * kXStageBytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kXStages + s); };
    const uint32_t acc_full = bar0 + 8u * (2 * kXStages);
    const uint32_t acc_empty = bar0 + 8u * (2 * kXStages + 1);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kXStages + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    double* epi = reinterpret_cast<double*>(base_ptr + kXStages * kXStageBytes + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = prm.k_pad / kXKB;
    const int tiles_n = (prm.n + kXTN - 1) / kXTN, tiles_m = (prm.m + kXTM - 1) / kXTM;
    const int num_tiles = tiles_m * tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kXStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 128);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int armed[kXStages];
#pragma unroll
            for (int s = 0; s < kXStages; ++s) armed[s] = -1;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int bi = tile / tiles_n, bj = tile - bi * tiles_n;
                int kb0, kb1;
                if (!x_tile_range(prm, bi, bj, nkb, kb0, kb1)) continue;
                for (int kb = kb0; kb < kb1 && ok; ++kb) {
                    ok = mbar_wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag);
                    if (!ok) break;
                    const uint32_t sbase = base + stage * kXStageBytes;
                    mbar_arrive_expect_tx(full_bar(stage), kXStageBytes);
                    armed[stage] = (int)phase;
#pragma unroll
                    for (int s = 0; s < kXSlices; ++s) {
                        tma_load_3d(sbase + s * kXABytes, &tmapA, kb * kXKB, bi * kXTM, s, full_bar(stage));
                        tma_load_3d(sbase + kXSlices * kXABytes + s * kXBBytes, &tmapB, kb * kXKB, bj * kXTN, s,
                                    full_bar(stage));
                    }
                    if (++stage == kXStages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // drain: wait (bounded) until the copies already issued have landed
                for (int s = 0; s < kXStages; ++s)
                    if (armed[s] >= 0) {
                        const long long t0 = clock64();
                        while (!mbar_try_wait(full_bar(s), (uint32_t)armed[s]) && clock64() - t0 < 200000000LL) {}
                    }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int bi = tile / tiles_n, bj = tile - bi * tiles_n;
                int kb0, kb1;
                if (!x_tile_range(prm, bi, bj, nkb, kb0, kb1)) continue;
                ok = mbar_wait_bounded(acc_empty, acc_phase ^ 1u, abort_flag);   // epilogue has drained TMEM
                if (!ok) break;
                tc_fence_after();
                for (int kb = kb0; kb < kb1 && ok; ++kb) {
                    ok = mbar_wait_bounded(full_bar(stage), phase, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sb = kDescLo + ((base + stage * kXStageBytes) >> 4);
                    const uint32_t first = kb > kb0 ? 1u : 0u;    // the first product of a group overwrites
#pragma unroll
                    for (int g = 0; g < kXGroups; ++g) {
#pragma unroll
                        for (int a = 0; a <= g; ++a) {
                            const int b = g - a;
#pragma unroll
                            for (int ks = 0; ks < kXKB / 32; ++ks) {
                                const uint32_t alo = sb + (uint32_t)((a * kXABytes) >> 4) + (uint32_t)(ks * 2);
                                const uint32_t blo = sb + (uint32_t)((kXSlices * kXABytes + b * kXBBytes) >> 4) +
                                                     (uint32_t)(ks * 2);
                                tc_mma_i8_lohi(tmem_base + g * kXTN, alo, blo, kDescHi, kGramIdesc,
                                               (a > 0 || ks > 0) ? 1u : first);
                            }
                        }
                    }
                    tc_commit(empty_bar(stage));     // the stage may be refilled once these MMAs have read it
                    if (++stage == kXStages) { stage = 0; phase ^= 1u; }
                }
                if (ok) tc_commit(acc_full);         // accumulators complete
                acc_phase ^= 1u;
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (warps 2..5)
        const int quarter = warp & 3;                 // TMEM lanes this warp may read
        const int r_in_tile = quarter * 32 + lane;
        double* my = epi + quarter * 32 * 17;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            const int bi = tile / tiles_n, bj = tile - bi * tiles_n;
            int kb0, kb1;
            if (!x_tile_range(prm, bi, bj, nkb, kb0, kb1)) {
                if (prm.out_mode == X_OUT_REDUCE && threadIdx.x == 64) prm.partials[tile] = 0.0;
                continue;
            }
            ok = mbar_wait_bounded(acc_full, acc_phase, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const int row = bi * kXTM + r_in_tile;
            // 1. drain: v = hi 2^32 + lo with lo = G6 + 2^8 G5 + 2^16 G4 + 2^24 G3, hi = G2 + 2^8 G1 + 2^16 G0, both exact
            double v[kXTN];
#pragma unroll
            for (int ch = 0; ch < kXTN / 16; ++ch) {
                long long lo[16], hi[16];
                uint32_t r[16];
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + ch * 16;
                tc_ld16(taddr + 6 * kXTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) lo[c] = (long long)(int)r[c];
                tc_ld16(taddr + 5 * kXTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) lo[c] += (long long)(int)r[c] << 8;
                tc_ld16(taddr + 4 * kXTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) lo[c] += (long long)(int)r[c] << 16;
                tc_ld16(taddr + 3 * kXTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) lo[c] += (long long)(int)r[c] << 24;
                tc_ld16(taddr + 2 * kXTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) hi[c] = (long long)(int)r[c];
                tc_ld16(taddr + 1 * kXTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) hi[c] += (long long)(int)r[c] << 8;
                tc_ld16(taddr + 0 * kXTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) hi[c] += (long long)(int)r[c] << 16;
#pragma unroll
                for (int c = 0; c < 16; ++c) v[ch * 16 + c] = fma((double)hi[c], 4294967296.0, (double)lo[c]);
            }
            tc_fence_before();
            mbar_arrive(acc_empty);
            acc_phase ^= 1u;
            // 2. C += alpha v 2^(48 - sh_i - sh_j), sixteen columns at a time through a transpose in shared memory:
            //    lane r writes its row's sixteen values, then half a warp reads one row's sixteen columns (128 bytes)
            const int sh_i = row < prm.m ? prm.sh_a[row] : 0;
            const double fi = prm.alpha * __longlong_as_double((long long)(1023 + 24 - sh_i) << 52);
            const int orow = lane >> 4, ocol = lane & 15;
            if (prm.out_mode == X_OUT_REDUCE) {
                // sum_ij P_ij D_ij over the tile, in a fixed order: along the row in this lane, then over the lanes of
                // the warp by a shuffle tree, then over the four warps in ascending order
                double s = 0.0;
                if (row < prm.m) {
                    const double* drow = prm.D + (int64_t)row * prm.ldd + bj * kXTN;
#pragma unroll
                    for (int c = 0; c < kXTN; ++c) {
                        const int col = bj * kXTN + c;
                        if (col < prm.n) {
                            const double fj = __longlong_as_double((long long)(1023 + 24 - prm.sh_b[col]) << 52);
                            s = fma((v[c] * fi) * fj, drow[c], s);
                        }
                    }
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
                if (lane == 0) my[0] = s;
                asm volatile("bar.sync 1, 128;" ::: "memory");           // the four epilogue warps
                if (quarter == 0 && lane == 0)
                    prm.partials[tile] = ((epi[0] + epi[32 * 17]) + epi[2 * 32 * 17]) + epi[3 * 32 * 17];
                asm volatile("bar.sync 1, 128;" ::: "memory");
                continue;
            }
            if (prm.out_mode == X_OUT_SYM) {
                // mirrored entries C[col][row]: consecutive lanes are consecutive rows, i.e. contiguous there
                if (row < prm.m) {
#pragma unroll
                    for (int c = 0; c < kXTN; ++c) {
                        const int col = bj * kXTN + c;
                        if (col < prm.n) {
                            const double fj = __longlong_as_double((long long)(1023 + 24 - prm.sh_b[col]) << 52);
                            prm.C[(int64_t)col * prm.ldc + row] = (v[c] * fi) * fj;
                        }
                    }
                }
            }
#pragma unroll
            for (int ch = 0; ch < kXTN / 16; ++ch) {
                const int col0 = bj * kXTN + ch * 16;
#pragma unroll
                for (int c = 0; c < 16; ++c) my[lane * 17 + c] = v[ch * 16 + c] * fi;
                __syncwarp();
                const int col = col0 + ocol;
                if (col < prm.n) {
                    const double fj = __longlong_as_double((long long)(1023 + 24 - prm.sh_b[col]) << 52);
                    double* dst0 = prm.C + (int64_t)(bi * kXTM + quarter * 32 + orow) * prm.ldc + col;
                    const int rows_left = prm.m - (bi * kXTM + quarter * 32 + orow);      // rows rr with rr < rows_left exist
                    // all sixteen old values are requested before the first is used: one memory latency per chunk
                    double oldv[16];
#pragma unroll
                    for (int q = 0; q < 16; ++q)
                        oldv[q] = (prm.out_mode != X_OUT_SYM && 2 * q < rows_left)
                                      ? __ldcg(dst0 + (int64_t)(2 * q) * prm.ldc) : 0.0;
#pragma unroll
                    for (int q = 0; q < 16; ++q)
                        if (2 * q < rows_left)
                            __stcg(dst0 + (int64_t)(2 * q) * prm.ldc, oldv[q] + my[(2 * q + orow) * 17 + ocol] * fj);
                }
                __syncwarp();
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
    if (threadIdx.x == 0 && *abort_flag) report(prm.status, PTQ_ERR_TIMEOUT, blockIdx.x, 4);
}

// ------------------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------------------
inline int x_make_map(CUtensorMap* m, int8_t* Q, int rows_pad, int k_pad, int box_rows) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return PTQ_ERR_CUDA;
    const cuuint64_t dims[3] = {(cuuint64_t)k_pad, (cuuint64_t)rows_pad, (cuuint64_t)kXSlices};
    const cuuint64_t strides[2] = {(cuuint64_t)k_pad, (cuuint64_t)rows_pad * (cuuint64_t)k_pad};
    const cuuint32_t box[3] = {(cuuint32_t)kXKB, (cuuint32_t)box_rows, 1u};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, Q, dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PTQ_OK : PTQ_ERR_CUDA;
}

// Slices of one operand in the workspace: planes [7][rows_pad][k_pad] and the per-row shifts.
struct XOperand {
    int8_t* Q;
    int32_t* sh;
    int rows, k;
};
inline size_t x_operand_bytes(int rows, int k) {
    return align_up(i8gemm_plane_bytes(rows, k)) + align_up((size_t)(cdiv(rows, 128) * 128) * sizeof(int32_t)) +
           align_up((size_t)(cdiv(rows, 128) * 128) * sizeof(unsigned long long));
}
// X is [rows x k] (transposed = 0, row stride ld) or [k x rows] (transposed = 1: the operand's rows are X's columns).
inline XOperand x_slice_operand(Carver& cv, const double* X, int64_t ld, int transposed, int rows, int k,
                                cudaStream_t stream) {
    const int rows_pad = cdiv(rows, 128) * 128, k_pad = cdiv(k, 128) * 128;
    XOperand op;
    op.Q = cv.take<int8_t>(i8gemm_plane_bytes(rows, k));
    op.sh = cv.take<int32_t>(rows_pad);
    unsigned long long* colmax = cv.take<unsigned long long>(rows_pad);
    op.rows = rows; op.k = k;
    Launch l(K_X_SLICE, stream);
    if (transposed) {
        cudaMemsetAsync(colmax, 0, (size_t)rows_pad * sizeof(unsigned long long), stream);
        x_colmax_kernel<<<dim3(rows_pad / 32, cdiv(k, kXColChunk)), 256, 0, stream>>>(X, k, rows, ld, colmax);
        x_slice_cols_kernel<<<dim3(rows_pad / 32, cdiv(k_pad, kXColChunk)), 256, 0, stream>>>(X, k, rows, ld, rows_pad, k_pad,
                                                                                              colmax, op.Q, op.sh);
    } else {
        x_slice_rows_kernel<<<rows_pad, 256, 0, stream>>>(X, rows, k, ld, rows_pad, k_pad, op.Q, op.sh);
    }
    return op;
}

// The product of two sliced operands (A: m rows, B: n rows, same k <= kXMaxK) in the given output / K-range modes.
inline int x_product(const XOperand& a, const XOperand& b, XGemmParams prm, cudaStream_t stream) {
    if (a.k != b.k || a.k > kXMaxK) return PTQ_ERR_UNSUPPORTED;
    DeviceState* dev = nullptr;
    int st = current_device_state(&dev);
    if (st) return st;
    st = ensure_smem_attr(dev, SA_XGEMM, [] {
        return cudaFuncSetAttribute(i8gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kXSmemBytes);
    });
    if (st) return st;
    const int k_pad = cdiv(a.k, 128) * 128;
    CUtensorMap mapA, mapB;
    st = x_make_map(&mapA, a.Q, cdiv(a.rows, 128) * 128, k_pad, kXTM);
    if (st) return st;
    st = x_make_map(&mapB, b.Q, cdiv(b.rows, 128) * 128, k_pad, kXTN);
    if (st) return st;
    prm.m = a.rows; prm.n = b.rows; prm.k_pad = k_pad;
    prm.sh_a = a.sh; prm.sh_b = b.sh;
    const int tiles = cdiv(prm.m, kXTM) * cdiv(prm.n, kXTN);
    const int grid = tiles < dev->sms ? tiles : dev->sms;
    {
        Launch l(K_X_GEMM, stream);
        i8gemm_kernel<<<grid, kXThreads, kXSmemBytes, stream>>>(mapA, mapB, prm);
    }
    return launch_status();
}
inline int x_num_tiles(int m, int n) { return cdiv(m, kXTM) * cdiv(n, kXTN); }

// C[m x n] += alpha * A B^T with A [m x k] (rows contiguous in k, stride lda) and B given either as [n x k]
// (b_is_kn = 0, stride ldb) or as [k x n] (b_is_kn = 1: B^T is what is stored, stride ldb).  k <= kXMaxK.
inline int i8gemm_nt(double* C, int64_t ldc, const double* A, int64_t lda, const double* B, int64_t ldb, int b_is_kn,
                     int m, int n, int k, double alpha, void* ws, int32_t* status, cudaStream_t stream) {
    if (m <= 0 || n <= 0 || k <= 0) return PTQ_OK;
    if (k > kXMaxK) return PTQ_ERR_UNSUPPORTED;
    Carver cv(ws);
    const XOperand a = x_slice_operand(cv, A, lda, 0, m, k, stream);
    const XOperand b = x_slice_operand(cv, B, ldb, b_is_kn, n, k, stream);
    XGemmParams prm{};
    prm.C = C; prm.ldc = ldc; prm.alpha = alpha; prm.status = status;
    prm.out_mode = X_OUT_ADD; prm.k_mode = X_K_ALL;
    return x_product(a, b, prm, stream);
}

}  // namespace ptq
