// Float64 blocked factorisation pieces: A = U^T U (upper Cholesky, in place, row-major), the inverse of the
// factor W = U^-T from the same sweep, and Hinv = W^T W.  Sec. 5 item 1 of the paper (Cholesky, then the inverse of
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

// A = H + lambda I, from each row's 64-column diagonal tile on (the factorisation reads the upper triangle only, whole
// tiles on the diagonal); one grid row per matrix row.
__global__ void damp_copy_kernel(const double* __restrict__ H, double* __restrict__ A, int n,
                                 const double* __restrict__ lambda) {
    const int i = blockIdx.y;
    const double lam = *lambda;
    const int64_t row = (int64_t)i * n;
    for (int j = (i & ~(kNB - 1)) + blockIdx.x * blockDim.x + threadIdx.x; j < n; j += gridDim.x * blockDim.x)
        A[row + j] = H[row + j] + (i == j ? lam : 0.0);
}

// ------------------------------------------------------------------------------------------------------------
// Blocked upper Cholesky A = U^T U as ONE persistent cooperative kernel (one CTA per SM, 256 threads).
// For each 64-row block k:
//   strip phase    every CTA that owns a 64-column panel chunk factorises the 64 x 64 diagonal block itself (all
//                  CTAs do the same arithmetic on it, so no broadcast is needed) and applies the same row
//                  operations to its chunk: the unblocked algorithm on a 64 x 128 strip, eight pivots at a time
//                  (see chol_strip).  That replaces "factor the block, then solve the panel against it".
//   trailing phase A[i][j] -= U[k][i]^T U[k][j] on the upper 64 x 64 tiles, float64 tensor-core MMA, operands
//                  double-buffered through shared memory with cp.async.
// When the next block row has few strip work items, a few CTAs update and factorise it (look-ahead) while the others
// are still applying the current one to the rows below, which takes the strip off the critical path.
// The phases are separated by a grid-wide barrier whose wait is bounded: when it expires the CTA records
// PTQ_ERR_TIMEOUT, raises the abort word and leaves; the other CTAs see the abort word and leave too.
// A non-positive or non-finite pivot is reported (PTQ_ERR_NOT_SPD, pivot index) and replaced by 1.
// ------------------------------------------------------------------------------------------------------------
constexpr int kCholThreads = 256;
constexpr int kCholLd = kNB + 4;                               // operand row stride (68 = 4 mod 16: conflict-free)
constexpr size_t kCholSmemBytes = sizeof(double) * (2 * 2 * kNB * kCholLd) + 16;

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// bar[0]: arrival counter (monotonic, zero at launch), bar[1]: abort word.  Returns false when the CTA must leave.
// spin_limit: SM clock cycles after which the wait gives up.
__device__ __forceinline__ bool grid_barrier(unsigned* bar, unsigned target, int* s_flag, long long spin_limit) {
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
                if (clock64() - t0 > spin_limit) { atomicExch(&bar[1], 1u); ok = 0; break; }
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

// Loads the 64 x ncols block A[r0 .. r0+63][c0 .. c0+ncols-1] into dst[64][kCholLd], ncols = 1 << lg in {16, 32, 64};
// entries beyond n are zero.  Every thread copies a fixed column (pair) of successive row groups, so a block that lies
// inside the matrix needs one pointer increment per copy and no bounds test.
// NT threads take part (the first NT of the CTA): all of them, or the first four warps when the other four are to
// go on computing meanwhile.
template <int NT = kCholThreads>
__device__ __forceinline__ void chol_load_block(double* dst, const double* __restrict__ A, int64_t ld, int n, int r0,
                                                int c0, int lg, int vec16) {
    if (NT < kCholThreads && threadIdx.x >= NT) return;
    const bool interior = r0 + kNB <= n && c0 + (1 << lg) <= n;
    if (vec16) {
        const int sh = lg - 1;                           // pairs per row = 1 << sh
        const int c = (threadIdx.x & ((1 << sh) - 1)) * 2;
        const int rstep = NT >> sh;
        int r = threadIdx.x >> sh;
        const double* src = A + (int64_t)(r0 + r) * ld + c0 + c;
        double* d = dst + r * kCholLd + c;
        if (interior) {
            for (; r < kNB; r += rstep, src += (int64_t)rstep * ld, d += rstep * kCholLd) cp_async16_cg(d, src, true);
        } else {
            for (; r < kNB; r += rstep, src += (int64_t)rstep * ld, d += rstep * kCholLd) {
                const bool ok = r0 + r < n && c0 + c < n;  // n is even on this path: a pair never straddles n
                cp_async16_cg(d, ok ? src : A, ok);
            }
        }
    } else {
        const int c = threadIdx.x & ((1 << lg) - 1);
        const int rstep = NT >> lg;
        int r = threadIdx.x >> lg;
        const double* src = A + (int64_t)(r0 + r) * ld + c0 + c;
        double* d = dst + r * kCholLd + c;
        for (; r < kNB; r += rstep, src += (int64_t)rstep * ld, d += rstep * kCholLd) {
            const bool ok = interior || (r0 + r < n && c0 + c < n);
            cp_async8(d, ok ? src : A, ok);
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
// Strip factorisation: the 64 x 128 strip [diagonal block | 64 panel columns] is held in registers as 8 x 8
// MMA accumulator fragments (warp w owns strip columns 16 w .. 16 w + 15, all 64 rows).  Pivots are taken eight
// at a time.  For pivot block b:
//   1. warp 0 factorises the 8 x 8 diagonal mini-block M = U_M^T U_M (all of M in every lane, so the serial chain of
//      eight pivots has no data exchange in it) and carries the identity along to obtain W = U_M^-T;
//   2. the new rows U[8 b .. 8 b + 7][:] = W R come from two MMAs per fragment (R: the row panel, published before);
//   3. they are published; every warp subtracts them from the rows of pivot block b + 1 FIRST and publishes those
//      rows at once, so that warp 0 can start on the next mini-block,
//   4. while the other warps subtract them from the rows further down, A[i][c] -= U[p][i] U[p][c], again by MMA.
// Warp 0 owns the first 16 columns of the diagonal block, whose fragments below row 16 are never used: it has no
// update work of its own in step 4 and is therefore the one that runs the chain.  Named barrier 1 hands the row panel
// to warp 0 (the others only arrive), named barrier 2 hands W to everybody.
// ------------------------------------------------------------------------------------------------------------
constexpr int kStripLd = 132;                                            // row stride of the 8-row panels
constexpr int kStripCostTiles = 4;                                       // a strip takes about as long as four trailing tiles
constexpr int kStripSmemDoubles = 2 * 8 * kStripLd + 64;
static_assert(kStripSmemDoubles <= 2 * 2 * kNB * kCholLd, "the strip panels alias the trailing-phase operand buffers");

__device__ __forceinline__ void strip_bar_sync(int id) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(kCholThreads) : "memory");
}
__device__ __forceinline__ void strip_bar_arrive(int id) {
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(kCholThreads) : "memory");
}

// Rows of pivot block B of this warp's columns go to the row panel.
template <int B>
__device__ __forceinline__ void chol_strip_publish(const double (&acc)[8][2][2], double* Rbuf, int c0, int lq, int lr) {
#pragma unroll
    for (int cb = 0; cb < 2; ++cb)
        *reinterpret_cast<double2*>(Rbuf + lq * kStripLd + c0 + 8 * cb + 2 * lr) =
            make_double2(acc[B][cb][0], acc[B][cb][1]);
}

// acc[r] -= U[:, 8 r .. 8 r + 7]^T U[:, own columns] for the fragment rows R0 <= r < R1 (U: the eight rows in Ubuf).
template <int R0, int R1>
__device__ __forceinline__ void chol_strip_update(double (&acc)[8][2][2], const double* Ubuf, int warp, int c0, int lq,
                                                  int lr) {
    if constexpr (R0 < R1) {
        double bf[2][2];
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
            bf[cb][0] = Ubuf[lr * kStripLd + c0 + 8 * cb + lq];
            bf[cb][1] = Ubuf[(4 + lr) * kStripLd + c0 + 8 * cb + lq];
        }
#pragma unroll
        for (int r = R0; r < R1; ++r) {
            const double n0 = -Ubuf[lr * kStripLd + 8 * r + lq];
            const double n1 = -Ubuf[(4 + lr) * kStripLd + 8 * r + lq];
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                if (warp < 4 && 8 * r > c0 + 8 * cb + 7) continue;       // entirely below the diagonal: never used
                dmma_884(acc[r][cb][0], acc[r][cb][1], n0, bf[cb][0]);
                dmma_884(acc[r][cb][0], acc[r][cb][1], n1, bf[cb][1]);
            }
        }
    }
}

// Look-ahead update of fragment row RB of this warp's strip columns with the block row above (see chol_strip):
//     acc[RB] -= ua[:, 8 RB .. 8 RB + 7]^T bsrc[:, own 16 columns]        (ua, bsrc: 64 x 64 in shared memory)
// Applied one fragment row at a time, just before the row is needed, by the warps that wait for warp 0's chain.
template <int RB>
__device__ __forceinline__ void chol_strip_lookahead(double (&acc)[8][2][2], const double* ua, const double* bsrc,
                                                     bool is_diag, int sc0, int lq, int lr) {
    double prod[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
#pragma unroll 4
    for (int kk = 0; kk < kNB; kk += 4) {
        const double af = ua[(kk + lr) * kCholLd + 8 * RB + lq];
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
            // fragments of the diagonal block that lie entirely below the diagonal are never used
            if (is_diag && 8 * RB > sc0 + 8 * cb + 7) continue;
            dmma_884(prod[cb][0], prod[cb][1], af, bsrc[(kk + lr) * kCholLd + 8 * cb + lq]);
        }
    }
#pragma unroll
    for (int cb = 0; cb < 2; ++cb) {
        acc[RB][cb][0] -= prod[cb][0];
        acc[RB][cb][1] -= prod[cb][1];
    }
}

template <int B>
__device__ __forceinline__ void chol_strip_block(double (&acc)[8][2][2], double* Rbuf, double* Ubuf, double* Wbuf,
                                                 int warp, int lane, int k0, bool reporter, int32_t* status,
                                                 const double* ua, const double* bsrc) {
    const int lq = lane >> 2, lr = lane & 3;
    const int c0 = 16 * warp;
    if (warp == 0) {
        // 1. the mini-block; lane j carries column j of the identity along, which becomes column j of W = U_M^-T
        double m[8][8];
#pragma unroll
        for (int p = 0; p < 8; ++p)
#pragma unroll
            for (int j = p; j < 8; ++j) m[p][j] = Rbuf[p * kStripLd + 8 * B + j];
        const int jc = lane & 7;
        double x[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) x[i] = i == jc ? 1.0 : 0.0;
        int bad = -1;                    // first pivot of this mini-block that is not positive and finite
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            // A bad pivot is replaced by 1 and remembered; the report is made after the chain, so that the eight steps
            // stay one straight line of code.
            const double d0 = m[p][p];
            const bool ok = d0 > 0.0 && d0 < 1.0e300;
            bad = (!ok && bad < 0) ? p : bad;
            const double d = ok ? d0 : 1.0;
            // 1 / sqrt(d): the hardware's approximation (about 20 bits) refined without a branch by
            // y (1 + e / 2 + 3 e^2 / 8), e = 1 - d y^2, which leaves an error of order e^3, far below one ulp;
            // the library routine is three times as long a chain
            double y;
            asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(d));
            const double e = fma(-(y * y), d, 1.0);
            const double rs = fma(y, e * fma(0.375, e, 0.5), y);
            const double inv = rs * rs;
            const double tx = x[p] * inv;
            x[p] *= rs;
#pragma unroll
            for (int i = p + 1; i < 8; ++i) {
                const double f = m[p][i] * inv;
                x[i] = fma(-m[p][i], tx, x[i]);
#pragma unroll
                for (int j = i; j < 8; ++j) m[i][j] = fma(-f, m[p][j], m[i][j]);
            }
        }
        if (lane < 8) {
#pragma unroll
            for (int p = 0; p < 8; ++p) Wbuf[p * 8 + lane] = x[p];    // W[p][j] = (U_M^-T)[p][j]
        }
        if (bad >= 0 && reporter) report(status, PTQ_ERR_NOT_SPD, k0 + 8 * B + bad);
    } else {
        // while warp 0 is in its chain: 4. (of the mini-block before) the rows further down, and the look-ahead update
        // of the rows of the next pivot block, which are needed right after this mini-block
        if constexpr (B > 0) chol_strip_update<B + 1, 8>(acc, Ubuf, warp, c0, lq, lr);
        if constexpr (B < 7) {
            if (bsrc != nullptr) chol_strip_lookahead<B + 1>(acc, ua, bsrc, warp < 4, c0, lq, lr);
        }
    }
    strip_bar_sync(2);       // W is there; nobody reads the previous new rows any more
    // 2. new rows = W R
    const double a0 = Wbuf[lq * 8 + lr], a1 = Wbuf[lq * 8 + 4 + lr];
#pragma unroll
    for (int cb = 0; cb < 2; ++cb) {
        const double b0 = Rbuf[lr * kStripLd + c0 + 8 * cb + lq];
        const double b1 = Rbuf[(4 + lr) * kStripLd + c0 + 8 * cb + lq];
        double r0 = 0.0, r1 = 0.0;
        dmma_884(r0, r1, a0, b0);
        dmma_884(r0, r1, a1, b1);
        acc[B][cb][0] = r0;
        acc[B][cb][1] = r1;
        *reinterpret_cast<double2*>(Ubuf + lq * kStripLd + c0 + 8 * cb + 2 * lr) = make_double2(r0, r1);
    }
    __syncthreads();
    // 3. the rows of the next pivot block first, and out they go
    if constexpr (B < 7) {
        chol_strip_update<B + 1, B + 2>(acc, Ubuf, warp, c0, lq, lr);
        chol_strip_publish<B + 1>(acc, Rbuf, c0, lq, lr);
        if (warp == 0) strip_bar_sync(1); else strip_bar_arrive(1);
    }
}
template <int... Bs>
__device__ __forceinline__ void chol_strip_blocks(double (&acc)[8][2][2], double* Rbuf, double* Ubuf, double* Wbuf,
                                                  int warp, int lane, int k0, bool reporter, int32_t* status,
                                                  const double* ua, const double* bsrc,
                                                  std::integer_sequence<int, Bs...>) {
    chol_strip_publish<0>(acc, Rbuf, 16 * warp, lane >> 2, lane & 3);
    if (warp == 0) strip_bar_sync(1); else strip_bar_arrive(1);
    (chol_strip_block<Bs>(acc, Rbuf, Ubuf, Wbuf, warp, lane, k0, reporter, status, ua, bsrc), ...);
}

// Factorises the diagonal block of A at k0 and applies the same row operations to 64 panel columns with it: columns
// pc0 .. pc0 + 63 of rows k0 .. k0 + 63 of the matrix P (row stride ld), or, when `identity` is set, of the identity
// block (whose transform is the inverse of the transposed diagonal factor).  P == nullptr: diagonal block only.
// Every CTA working on this block row reads the diagonal block of A, at a time of its own, so the factor of that
// block is NOT written in place: the CTA with write_diag set stores it to D (64 x 64, row stride 64), and the kernel
// copies all diagonal factors into A at its very end.
// When upd_a is given, the strip is first brought up to date with the previous block row (look-ahead):
//     strip -= upd_a^T [upd_a | upd_b],   upd_a[kk][r] = U[k0 - 64 + kk][k0 + r],  upd_b[kk][c] = P[k0 - 64 + kk][pc0 + c]
// (both 64 x 64 in shared memory, row stride kCholLd; upd_b == nullptr: the panel part needs no update).
__device__ __forceinline__ void chol_strip(double* __restrict__ A, int64_t ld, int n, int k0, double* __restrict__ P,
                                           int pc0, bool identity, bool write_diag, double* __restrict__ D,
                                           double* smem, int vec16, int32_t* status, const double* upd_a,
                                           const double* upd_b) {
    // "warp" below is the index of the 16-column group a warp owns, not its hardware number.  Warps w and w + 4 share a
    // scheduler; warp 0 (group 0, the chain) is paired with the next lightest group (diagonal columns 16 .. 31, whose
    // fragments below row 32 are unused) and the heavier groups are spread over the other schedulers:
    // hardware warp 0 1 2 3 4 5 6 7 -> group 0 2 3 6 1 4 5 7.
    const int lane = threadIdx.x & 31, warp = (int)((0x75416320u >> (4 * (threadIdx.x >> 5))) & 7u);
    const int lq = lane >> 2, lr = lane & 3;
    double* Rbuf = smem;
    double* Ubuf = smem + 8 * kStripLd;
    double* Wbuf = smem + 2 * 8 * kStripLd;
    const bool is_diag = warp < 4;
    const int gc0 = is_diag ? k0 + 16 * warp : pc0 + 16 * (warp - 4);       // first global column of this warp
    const int sc0 = 16 * warp;                                               // first strip column
    double acc[8][2][2];
    // panel columns that lie inside the matrix and are not the identity: plain vector loads
    const bool fast_panel = !is_diag && P != nullptr && !identity && vec16 && k0 + kNB <= n && pc0 + kNB <= n;
    if (fast_panel) {
        const double* src = P + (int64_t)(k0 + lq) * ld + gc0 + 2 * lr;
#pragma unroll
        for (int rb = 0; rb < 8; ++rb)
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                const double2 v = __ldcg(reinterpret_cast<const double2*>(src + (int64_t)(8 * rb) * ld + 8 * cb));
                acc[rb][cb][0] = v.x;
                acc[rb][cb][1] = v.y;
            }
    } else {
#pragma unroll
        for (int rb = 0; rb < 8; ++rb)
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                const int row = 8 * rb + lq, grow = k0 + row;
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int sc = sc0 + 8 * cb + 2 * lr + e, gc = gc0 + 8 * cb + 2 * lr + e;
                    double val = 0.0;
                    if (is_diag) {
                        if (sc >= row) {
                            if (grow < n && gc < n) val = __ldcg(A + (int64_t)grow * ld + gc);
                            else if (sc == row) val = 1.0;                   // identity padding below n
                        }
                    } else if (P != nullptr && grow < n && gc < n) {
                        val = identity ? (sc - kNB == row ? 1.0 : 0.0) : __ldcg(P + (int64_t)grow * ld + gc);
                    }
                    acc[rb][cb][e] = val;
                }
            }
    }
    // Look-ahead update with the block row above: only the first fragment row (and warp 0's second: warp 0 runs the
    // chains and has no other rows in use) is brought up to date here; the others follow inside the strip, each while
    // warp 0 works on the mini-block before it.
    const double* bsrc = nullptr;
    if (upd_a != nullptr) {
        cp_async_wait<0>();
        __syncthreads();
        bsrc = is_diag ? upd_a + 16 * warp : (upd_b != nullptr ? upd_b + 16 * (warp - 4) : nullptr);
        if (bsrc != nullptr) {
            chol_strip_lookahead<0>(acc, upd_a, bsrc, is_diag, sc0, lq, lr);
            if (warp == 0) chol_strip_lookahead<1>(acc, upd_a, bsrc, is_diag, sc0, lq, lr);
        }
    }
    chol_strip_blocks(acc, Rbuf, Ubuf, Wbuf, warp, lane, k0, write_diag && threadIdx.x == 0, status, upd_a, bsrc,
                      std::make_integer_sequence<int, 8>());
    if (is_diag) {
        if (write_diag) {
#pragma unroll
            for (int rb = 0; rb < 8; ++rb)
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    const int row = 8 * rb + lq, sc = sc0 + 8 * cb + 2 * lr;
                    if (sc >= row) D[row * kNB + sc] = acc[rb][cb][0];
                    if (sc + 1 >= row) D[row * kNB + sc + 1] = acc[rb][cb][1];
                }
        }
    } else if (P != nullptr) {
#pragma unroll
        for (int rb = 0; rb < 8; ++rb)
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                const int grow = k0 + 8 * rb + lq, gc = gc0 + 8 * cb + 2 * lr;
                if (grow >= n || gc >= n) continue;
                double* dst = P + (int64_t)grow * ld + gc;
                if (vec16) {
                    __stcg(reinterpret_cast<double2*>(dst), make_double2(acc[rb][cb][0], acc[rb][cb][1]));
                } else {
                    __stcg(dst, acc[rb][cb][0]);
                    if (gc + 1 < n) __stcg(dst + 1, acc[rb][cb][1]);
                }
            }
    }
}

// One H x 64 piece of a trailing tile: C[i0 .. i0 + H)[j0 .. j0 + 64) -= as^T bs with the operands in shared memory
// (as[kk][r], bs[kk][c]); eight warps as 2 x 4, each (H / 2) x 16.  tri_off >= 0: the piece lies in a diagonal tile
// and only entries with c >= tri_off + r are touched.
template <int H>
__device__ __forceinline__ void chol_trailing_piece(double* __restrict__ C, int64_t ld, int n, const double* as,
                                                    const double* bs, int i0, int j0, int tri_off, int vec16) {
    constexpr int FM = H / 16, FN = 2;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int wm0 = (warp >> 2) * (H / 2), wn0 = (warp & 3) * 16;
    const int lq = lane >> 2, lr = lane & 3;
    // the old values of the tile are requested first and only consumed after the MMA loop, so that their latency
    // hides behind it
    double old[FM][FN][2], acc[FM][FN][2];
    bool keep[FM][FN][2];
    // a piece inside the matrix and off the diagonal needs no bounds or triangle tests at all
    const bool plain = vec16 && tri_off < 0 && i0 + H <= n && j0 + kNB <= n;
    if (plain) {
        const double* src = C + (int64_t)(i0 + wm0 + lq) * ld + j0 + wn0 + 2 * lr;
#pragma unroll
        for (int a = 0; a < FM; ++a)
#pragma unroll
            for (int b = 0; b < FN; ++b) {
                const double2 v = __ldcg(reinterpret_cast<const double2*>(src + (int64_t)(8 * a) * ld + 8 * b));
                old[a][b][0] = v.x;
                old[a][b][1] = v.y;
                acc[a][b][0] = acc[a][b][1] = 0.0;
                keep[a][b][0] = keep[a][b][1] = true;
            }
    } else
#pragma unroll
    for (int a = 0; a < FM; ++a) {
        const int r = wm0 + a * 8 + lq;
#pragma unroll
        for (int b = 0; b < FN; ++b) {
            const int c = wn0 + b * 8 + 2 * lr;
            const bool in = i0 + r < n && j0 + c < n;
            keep[a][b][0] = in && (tri_off < 0 || c >= tri_off + r);
            keep[a][b][1] = in && j0 + c + 1 < n && (tri_off < 0 || c + 1 >= tri_off + r);
            const double* src = C + (int64_t)(i0 + r) * ld + j0 + c;
            if (vec16 && keep[a][b][0]) {             // n even: the pair is inside; keep[0] implies keep[1]
                const double2 v = __ldcg(reinterpret_cast<const double2*>(src));
                old[a][b][0] = v.x;
                old[a][b][1] = v.y;
            } else {
                old[a][b][0] = keep[a][b][0] ? __ldcg(src) : 0.0;
                old[a][b][1] = keep[a][b][1] ? __ldcg(src + 1) : 0.0;
            }
            acc[a][b][0] = acc[a][b][1] = 0.0;
        }
    }
#pragma unroll 4
    for (int kk = 0; kk < kNB; kk += 4) {
        double af[FM], bf[FN];
#pragma unroll
        for (int a = 0; a < FM; ++a) af[a] = as[(kk + lr) * kCholLd + wm0 + a * 8 + lq];
#pragma unroll
        for (int b = 0; b < FN; ++b) bf[b] = bs[(kk + lr) * kCholLd + wn0 + b * 8 + lq];
#pragma unroll
        for (int a = 0; a < FM; ++a)
#pragma unroll
            for (int b = 0; b < FN; ++b) dmma_884(acc[a][b][0], acc[a][b][1], af[a], bf[b]);
    }
    if (plain) {
        double* dst = C + (int64_t)(i0 + wm0 + lq) * ld + j0 + wn0 + 2 * lr;
#pragma unroll
        for (int a = 0; a < FM; ++a)
#pragma unroll
            for (int b = 0; b < FN; ++b)
                __stcg(reinterpret_cast<double2*>(dst + (int64_t)(8 * a) * ld + 8 * b),
                       make_double2(old[a][b][0] - acc[a][b][0], old[a][b][1] - acc[a][b][1]));
        return;
    }
#pragma unroll
    for (int a = 0; a < FM; ++a) {
        const int r = wm0 + a * 8 + lq;
#pragma unroll
        for (int b = 0; b < FN; ++b) {
            const int c = wn0 + b * 8 + 2 * lr;
            double* dst = C + (int64_t)(i0 + r) * ld + j0 + c;
            const double v0 = old[a][b][0] - acc[a][b][0], v1 = old[a][b][1] - acc[a][b][1];
            if (vec16 && keep[a][b][0]) {
                __stcg(reinterpret_cast<double2*>(dst), make_double2(v0, v1));
            } else {
                if (keep[a][b][0]) __stcg(dst, v0);
                if (keep[a][b][1]) __stcg(dst + 1, v1);
            }
        }
    }
}

__global__ void __launch_bounds__(kCholThreads, 1)
chol_coop_kernel(double* __restrict__ A, double* __restrict__ Wm, double* __restrict__ Dbuf, int n, int64_t ld,
                 int vec16, unsigned* bar, int32_t* status, long long spin_limit, int k_first, int nb_stop,
                 int row_limit) {
    extern __shared__ __align__(16) unsigned char chol_smem_raw[];
    double* opnd = reinterpret_cast<double*>(chol_smem_raw);                // [2 stages][2 operands][64][kCholLd]
    int* s_flag = reinterpret_cast<int*>(opnd + 2 * 2 * kNB * kCholLd);     // the strip panels alias opnd
    const int tid = threadIdx.x;
    const int G = gridDim.x;
    const int nb = (n + kNB - 1) / kNB;
    unsigned epoch = 0;

    // strip work items of block row k: the panel chunks of A right of the block, then (with Wm) the chunks 0 .. k of
    // row block k of W, the last of which starts as the identity
    auto strip_items = [&](int k) { return (nb - 1 - k) + (Wm != nullptr ? k + 1 : 0); };
    auto strip_item = [&](int k, int g, double*& P, int& pc0, bool& ident) {
        const int chunksA = nb - 1 - k;
        P = nullptr; pc0 = 0; ident = false;
        if (g < chunksA) { P = A; pc0 = (k + 1 + g) * kNB; }
        else if (g < strip_items(k)) { P = Wm; pc0 = (g - chunksA) * kNB; ident = (g - chunksA) == k; }
    };
    // plain strip phase of block row k over the whole grid
    auto strip_phase = [&](int k) {
        const int items = strip_items(k);
        const int reps = items > 0 ? items : 1;                              // last block without Wm: diagonal only
        for (int g = blockIdx.x; g < reps; g += G) {
            double* P; int pc0; bool ident;
            strip_item(k, g, P, pc0, ident);
            chol_strip(A, ld, n, k * kNB, P, pc0, ident, g == 0, Dbuf + (size_t)k * kNB * kNB, opnd, vec16, status, nullptr,
                       nullptr);
            __syncthreads();     // the panel buffers are reused by the next repetition and by the trailing phase
        }
    };
    // Trailing tiles of block row k restricted to the target block rows row_base <= i < row_limit.
    //   tiles of A: (i, j), row_base <= i <= j: A[i][j] -= U[k][i]^T U[k][j]
    //   tiles of W: (i, c), row_base <= i, c <= k:  W[i][c] -= U[k][i]^T W[k][c]       (row-major lists, A first)
    // In look-ahead mode the CTAs come here after `strips_b` strips of the next block row, the CTAs 0 .. n_more - 1 after
    // one more; a strip costs about as much as kStripCostTiles tiles, so they take correspondingly fewer pieces (the
    // busier CTAs from the end of the list) and all CTAs finish at about the same time.
    auto trailing_phase = [&](int k, int row_base, int n_more, int strips_b) {
        const int k0 = k * kNB;
        const int m = nb - row_base;                                        // tiles in the first target row
        const int R = (row_limit < nb ? row_limit : nb) - row_base;         // target block rows
        if (R <= 0) return;
        const int TA = R * m - R * (R - 1) / 2;
        const int TW = Wm != nullptr ? R * (k + 1) : 0;
        const int T = TA + TW;
        if (T <= 0) return;
        // tiles are cut into 64 / H row pieces so that a short tile list still spreads over the grid
        const int lgH = 4 * T <= G ? 4 : (2 * T <= G ? 5 : 6);
        const int lgP = 6 - lgH;
        const int TP = T << lgP;
        const int S = n_more < G ? n_more : G, N = G - S;
        const int cs = kStripCostTiles << lgP;
        const int cost_a = (strips_b + 1) * cs, cost_b = strips_b * cs;
        int ps = 0;
        if (S > 0) {
            const long work = (long)TP + (long)S * cost_a + (long)N * cost_b;
            const int target = (int)((work + G - 1) / G);
            ps = target > cost_a ? target - cost_a : 0;
            if (N == 0) ps = (TP + S - 1) / S;
        }
        const int TPn = TP - S * ps > 0 ? TP - S * ps : 0;
        const int pn = N > 0 ? (TPn + N - 1) / N : 0;
        int tp_beg, tp_end;
        if ((int)blockIdx.x >= S) {
            tp_beg = ((int)blockIdx.x - S) * pn;
            tp_end = tp_beg + pn < TPn ? tp_beg + pn : TPn;
        } else {
            tp_beg = TPn + (int)blockIdx.x * ps;
            tp_end = tp_beg + ps < TP ? tp_beg + ps : TP;
        }
        if (tp_beg >= tp_end) return;
        struct Piece { double* C; const double* Bsrc; int i0, j0, tri; };
        // pieces are asked for in ascending order, so the row of the triangular list is found by walking on from the
        // row of the previous piece
        int cur_r = 0, cur_start = 0;                       // row cur_r of the A list starts at tile cur_start
        auto piece_of = [&](int tp) {
            Piece pc;
            const int t = tp >> lgP;
            const int h0 = (tp & ((1 << lgP) - 1)) << lgH;
            if (t < TA) {
                while (t >= cur_start + (m - cur_r)) { cur_start += m - cur_r; ++cur_r; }
                const int r = cur_r;
                const int bi = row_base + r, bj = bi + (t - cur_start);
                pc.C = A; pc.Bsrc = A; pc.i0 = bi * kNB + h0; pc.j0 = bj * kNB;
                pc.tri = bi == bj ? h0 : -1;
            } else {
                const int tw = t - TA;
                const int r = tw / (k + 1), c = tw - r * (k + 1);
                pc.C = Wm; pc.Bsrc = Wm; pc.i0 = (row_base + r) * kNB + h0; pc.j0 = c * kNB;
                pc.tri = -1;
            }
            return pc;
        };
        // Operand blocks: slot s of the A half holds U[k][i-block] (as[kk][r]), slot s of the B half U or W [k][j-block].
        // Every CTA takes a contiguous run of the list, in which consecutive tiles mostly share their row block: the A
        // operand then stays where it is and only B is fetched.
        double* abuf = opnd;                                  // [2][64][kCholLd]
        double* bbuf = opnd + 2 * kNB * kCholLd;              // [2][64][kCholLd]
        int stage = 0, a_slot = 0, a_next = 0;
        Piece cur{}, nxt{};
        if (tp_beg < tp_end) {
            cur = piece_of(tp_beg);
            chol_load_block(abuf, A, ld, n, k0, cur.i0, lgH, vec16);
            chol_load_block(bbuf, cur.Bsrc, ld, n, k0, cur.j0, 6, vec16);
        }
        cp_async_commit();
        for (int tp = tp_beg; tp < tp_end; ++tp) {
            cp_async_wait<0>();
            __syncthreads();         // this tile's operands have landed; the slots of the tile before are free
            // The next tile's operands are requested by the first four warps only: the copies keep the issuing warps
            // busy for several hundred cycles, during which the other four (one per scheduler) already feed the
            // tensor pipe.
            if (tp + 1 < tp_end) {
                nxt = piece_of(tp + 1);
                a_next = a_slot;
                if (nxt.i0 != cur.i0) {
                    a_next = a_slot ^ 1;
                    chol_load_block<kCholThreads / 2>(abuf + a_next * kNB * kCholLd, A, ld, n, k0, nxt.i0, lgH, vec16);
                }
                chol_load_block<kCholThreads / 2>(bbuf + (stage ^ 1) * kNB * kCholLd, nxt.Bsrc, ld, n, k0, nxt.j0, 6,
                                                  vec16);
            }
            cp_async_commit();
            const double* as = abuf + a_slot * kNB * kCholLd;
            const double* bs = bbuf + stage * kNB * kCholLd;
            if (lgH == 6) chol_trailing_piece<64>(cur.C, ld, n, as, bs, cur.i0, cur.j0, cur.tri, vec16);
            else if (lgH == 5) chol_trailing_piece<32>(cur.C, ld, n, as, bs, cur.i0, cur.j0, cur.tri, vec16);
            else chol_trailing_piece<16>(cur.C, ld, n, as, bs, cur.i0, cur.j0, cur.tri, vec16);
            stage ^= 1;
            a_slot = a_next;
            cur = nxt;
        }
        cp_async_wait<0>();
    };

    // The block rows k_first .. nb_stop - 1 are factorised (block row k_first must already carry the updates of all rows
    // above it); their updates are applied to the target rows below row_limit.
    //   k_first = 0, nb_stop = nb, row_limit = nb : the whole factorisation;
    //   nb_stop < nb, row_limit = nb : a partial factorisation that leaves the Schur complement of the leading block in
    //       the upper triangle of A[64 nb_stop :, 64 nb_stop :] (what Eq. 12 leaves after that many columns);
    //   row_limit = nb_stop : a panel -- only its own block rows are touched; the caller applies the panel to the rows
    //       below it in one product of depth 64 (nb_stop - k_first).
    const int nbs = nb_stop < nb ? nb_stop : nb;
    const int steps = nbs < nb ? (row_limit > nbs ? nbs : nbs - 1) : nb - 1;
    strip_phase(k_first);
    for (int k = k_first; k < steps; ++k) {
        ++epoch;
        if (!grid_barrier(bar, epoch * (unsigned)G, s_flag, spin_limit)) break;
        // Block row k is final; the updates of block rows < k have been applied everywhere.
        if (k + 1 >= nbs) {                  // last factorised block row of a partial run: its update only
            trailing_phase(k, k + 1, 0, 0);
            continue;
        }
        const int next_items = strip_items(k + 1) > 0 ? strip_items(k + 1) : 1;
        // Look-ahead: the CTAs factorise the strips of block row k + 1 first (item g by CTA g mod G; each brings its
        // strip up to date with block row k itself) and then join the trailing tiles of block row k below row k + 1 with
        // a share reduced by what their strips cost, so nobody idles and there is one grid barrier per block row.
        for (int g = blockIdx.x; g < next_items; g += G) {
            double* P; int pc0; bool ident;
            strip_item(k + 1, g, P, pc0, ident);
            double* ua = opnd + 2 * kNB * kCholLd;        // beyond the strip's own panel buffers
            double* ub = ua + kNB * kCholLd;
            const bool need_b = P != nullptr && !ident;
            __syncthreads();
            chol_load_block(ua, A, ld, n, k * kNB, (k + 1) * kNB, 6, vec16);
            if (need_b) chol_load_block(ub, P, ld, n, k * kNB, pc0, 6, vec16);
            cp_async_commit();
            chol_strip(A, ld, n, (k + 1) * kNB, P, pc0, ident, g == 0, Dbuf + (size_t)(k + 1) * kNB * kNB, opnd, vec16,
                       status, ua, need_b ? ub : nullptr);
            __syncthreads();
        }
        trailing_phase(k, k + 2, next_items % G, next_items / G);
    }
    cp_async_wait<0>();
    // the diagonal factors move from the side buffer into A once nobody reads the original diagonal blocks any more
    ++epoch;
    if (grid_barrier(bar, epoch * (unsigned)G, s_flag, spin_limit)) {
        for (int b = k_first + blockIdx.x; b < nbs; b += G)
            for (int idx = tid; idx < kNB * kNB; idx += kCholThreads) {
                const int r = idx >> 6, c = idx & 63;
                if (c >= r && b * kNB + c < n)
                    A[(int64_t)(b * kNB + r) * ld + b * kNB + c] = __ldcg(Dbuf + (size_t)b * kNB * kNB + idx);
            }
    }
    if (tid == 0 && ld_acquire_u32(&bar[1]) != 0u) report(status, PTQ_ERR_TIMEOUT, blockIdx.x, 1);
}

// In-place blocked upper Cholesky A = U^T U of the n x n matrix A (row stride n).  Only the upper triangle is read or
// written.  With Wm (n x n, zero on entry) the same sweep also leaves W = U^-T there (lower triangular): the row
// operations of the factorisation are applied to the identity, which gives the inverse of the Cholesky factor that
// Sec. 5 item 1 asks for.
// `bar` is 2 x uint32 of device scratch, Dbuf holds chol_scratch_doubles(n) doubles (the diagonal factors on their way).
inline size_t chol_scratch_doubles(int n) { return (size_t)((n + kNB - 1) / kNB) * kNB * kNB; }
// nb_stop > 0: factorise the block rows k_first .. nb_stop - 1 only (see the kernel for what row_limit selects;
// row_limit <= 0: all rows below are updated).  A partial run that updates everything below must not ask for Wm.
inline int cholesky_upper(double* A, int n, double* Wm, double* Dbuf, unsigned* bar, int32_t* status,
                          cudaStream_t stream, int nb_stop = 0, int k_first = 0, int row_limit = 0) {
    const int nb_all = (n + kNB - 1) / kNB;
    if (nb_stop <= 0) nb_stop = nb_all;
    if (row_limit <= 0) row_limit = nb_all;
    if (nb_stop < nb_all && row_limit > nb_stop && Wm != nullptr) return PTQ_ERR_INVALID_ARG;
    if (k_first < 0 || k_first >= nb_stop) return PTQ_ERR_INVALID_ARG;
    DeviceState* dev = nullptr;
    int st = current_device_state(&dev);
    if (st) return st;
    if (!dev->coop) return PTQ_ERR_UNSUPPORTED;
    st = ensure_smem_attr(dev, SA_CHOL, [] {
        cudaError_t e = cudaFuncSetAttribute(chol_coop_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kCholSmemBytes);
        int per_sm = 0;
        if (e == cudaSuccess)
            e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, chol_coop_kernel, kCholThreads, kCholSmemBytes);
        return (e == cudaSuccess && per_sm < 1) ? cudaErrorLaunchOutOfResources : e;
    });
    if (st) return st;
    // One CTA per SM (the cooperative launch guarantees that all of them are resident); a matrix of a few block rows
    // gets only as many CTAs as it ever has work items, which makes its grid barriers cheaper and leaves SMs to kernels
    // of other streams.
    const int nbr = (n + kNB - 1) / kNB;
    const long items = (long)nbr * (nbr + 1) / 2 + (Wm != nullptr ? (long)nbr * nbr : 0);
    const int budget = coop_cta_budget(dev);
    const int grid = items < budget ? (int)(items < 1 ? 1 : items) : budget;
    if (cudaMemsetAsync(bar, 0, 2 * sizeof(unsigned), stream) != cudaSuccess) return PTQ_ERR_CUDA;
    int64_t ld = n;
    int vec16 = ((n & 1) == 0 && aligned16(A) && aligned16(Wm)) ? 1 : 0;
    long long spin_limit = kSpinLimitCycles;
    void* args[] = {&A, &Wm, &Dbuf, &n, &ld, &vec16, &bar, &status, &spin_limit, &k_first, &nb_stop, &row_limit};
    Launch l(K_CHOL_COOP, stream);
    if (cudaLaunchCooperativeKernel((const void*)chol_coop_kernel, dim3(grid), dim3(kCholThreads), args,
                                    kCholSmemBytes, stream) != cudaSuccess) {
        cudaGetLastError();
        return PTQ_ERR_CUDA;
    }
    return PTQ_OK;
}

// Hinv = W^T W for the lower-triangular W = U^-T: Hinv[i][j] = sum over k >= max(i, j) of W[k][i] W[k][j]; upper tiles
// computed, mirrored below.
inline int lauum_lower(const double* W, double* Hinv, int n, cudaStream_t stream) {
    GemmParams g = gemm_defaults();
    g.A = W; g.lda = n; g.a_trans = 1;
    g.B = W; g.ldb = n; g.b_trans = 0;
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
