// Float64 GEMM tile kernel used by every float64 stage: the triangular inverse, Hinv = V V^T, the float64
// cross-check Gram and the loss 1/2 tr(dW H dW^T).  One kernel, parameterised by operand layout and by the
// triangular structure it may exploit.  The products run on the float64 tensor-core instruction
// (mma.sync m8n8k4), operands are staged through shared memory by a 3-stage cp.async pipeline.
// All sums run over k in ascending order, so results are deterministic.
#pragma once
#include "common.cuh"

namespace ptq {

struct GemmParams {
    const double* A;   // a_trans == 0: A[i * lda + k]   a_trans == 1: A[k * lda + i]
    const double* B;   // b_trans == 0: B[k * ldb + j]   b_trans == 1: B[j * ldb + k]
    double* C;         // C[i * ldc + j] = alpha * sum_k A B + beta * C
    int64_t lda, ldb, ldc;
    int M, N, K;
    int a_trans, b_trans;
    double alpha, beta;
    int kbeg_mode;     // 0: k from 0;  1: from max(i0, j0);  2: from i0   (operands are zero before that)
    int kend_mode;     // 0: k to K;    1: to min(K, j0 + BN)              (B is zero after that)
    int sym_double;    // B symmetric, C not written (reduction epilogue): with kend_mode 1, the k blocks before the tile's
                       // own column block count twice, which stands in for the skipped blocks after it
    int upper_only;    // skip tiles that lie entirely below the diagonal
    int mirror;        // also store C[j][i] for tiles above the diagonal
    // batch z = blockIdx.z: operands advance by these element strides
    int64_t batch_a, batch_b, batch_c;
    int ragN_lim, ragN_step;   // if ragN_step > 0: N_z = min(N, ragN_lim - z * ragN_step)
    int k_is_n;                // K_z = N_z
    // optional reduction epilogue: partials[tile] = sum_ij acc_ij * D[i][j]; C is not written
    const double* D;
    int64_t ldd;
    double* partials;
    // ksplit > 1 (reduction epilogue only, one batch): blockIdx.z selects one of ksplit slices of the tile's k range;
    // every slice writes its own partial sum, which is all a sum over k needs
    int ksplit;
};

constexpr int kGemmBK = 32;
constexpr int kGemmStages = 3;
constexpr int kGemmThreads = 256;
constexpr int kGemmLdk = kGemmBK + 4;   // row stride of a k-contiguous operand tile (20 = 4 mod 16: conflict-free)

template <int BT>
constexpr int gemm_tile_doubles() { return BT * kGemmLdk; }   // >= 16 * (BT + 4), the m-contiguous layout
template <int BT>
constexpr size_t gemm_smem_bytes() { return size_t(kGemmStages) * 2 * gemm_tile_doubles<BT>() * sizeof(double); }

__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gsrc, bool valid) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const int sz = valid ? 8 : 0;    // src-size 0: the 8 bytes are filled with zeros
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(d), "l"(gsrc), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void dmma_884(double& c0, double& c1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c0), "+d"(c1)
                 : "d"(a), "d"(b));
}

// BT x BT output tile (bx, by) of batch z, 256 threads = 8 warps as 2 x 4; each warp owns (BT/2) x (BT/4) outputs as
// 8 x 8 fragments.  nbx = number of column tiles (indexes the partials).
template <int BT>
__device__ __forceinline__ void dgemm_tile(const GemmParams& p, int bx, int by, int z, int nbx, int nby) {
    constexpr int BK = kGemmBK;
    constexpr int LDM = BT + 4;            // row stride of an m-contiguous operand tile
    constexpr int TILE = BT * kGemmLdk;
    constexpr int WTM = BT / 2, WTN = BT / 4;
    constexpr int FM = WTM / 8, FN = WTN / 8;
    constexpr int EPT = BT * BK / kGemmThreads;
    extern __shared__ __align__(16) double smem[];

    int N = p.N, K = p.K;
    if (p.ragN_step > 0) {
        int lim = p.ragN_lim - z * p.ragN_step;
        if (lim < N) N = lim;
        if (N <= 0) return;
    }
    if (p.k_is_n) K = N;
    const int M = p.M;
    const int i0 = by * BT, j0 = bx * BT;
    if (i0 >= M || j0 >= N) return;
    if (p.upper_only && i0 >= j0 + BT) return;

    const double* __restrict__ A = p.A + z * p.batch_a;
    const double* __restrict__ B = p.B + z * p.batch_b;
    double* __restrict__ C = p.C ? p.C + z * p.batch_c : nullptr;

    int kbeg = 0, kend = K;
    if (p.kbeg_mode == 1) kbeg = (i0 > j0 ? i0 : j0);
    else if (p.kbeg_mode == 2) kbeg = i0;
    kbeg = (kbeg / BK) * BK;
    if (p.kend_mode == 1 && j0 + BT < kend) kend = j0 + BT;
    bool double_at_end = false;
    if (p.ksplit > 1) {
        const int len = ((kend - kbeg + BK - 1) / BK + p.ksplit - 1) / p.ksplit * BK;
        kbeg += z * len;
        if (kbeg + len < kend) kend = kbeg + len;
        // a slice that ends before the tile's own column block lies entirely in the part that counts twice
        double_at_end = p.sym_double && kend <= j0;
        z = 0;
    }
    const int zp = p.ksplit > 1 ? (int)blockIdx.z : z;          // index of the partial sum

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm0 = (warp >> 2) * WTM, wn0 = (warp & 3) * WTN;
    const int lq = lane >> 2, lr = lane & 3;
    const int a_trans = p.a_trans, b_trans = p.b_trans;

    double acc[FM][FN][2];
#pragma unroll
    for (int a = 0; a < FM; ++a)
#pragma unroll
        for (int b = 0; b < FN; ++b) acc[a][b][0] = acc[a][b][1] = 0.0;

    // operand tiles that lie inside their matrices are fetched two doubles at a time when the addresses allow it
    const bool a_vec = (reinterpret_cast<uintptr_t>(A) & 15u) == 0 && (p.lda & 1) == 0 && i0 + BT <= M;
    const bool b_vec = (reinterpret_cast<uintptr_t>(B) & 15u) == 0 && (p.ldb & 1) == 0 && j0 + BT <= N;
    auto load_stage = [&](int stage, int k0) {
        double* as = smem + (size_t)stage * 2 * TILE;
        double* bs = as + TILE;
        const bool kfull = k0 + BK <= kend;
        if (a_vec && kfull) {
#pragma unroll
            for (int r = 0; r < EPT / 2; ++r) {
                const int idx = tid + r * kGemmThreads;          // pair index
                if (a_trans == 0) {
                    const int k = (idx % (BK / 2)) * 2, m = idx / (BK / 2);
                    cp_async16(as + m * kGemmLdk + k, A + (int64_t)(i0 + m) * p.lda + k0 + k);
                } else {
                    const int m = (idx % (BT / 2)) * 2, k = idx / (BT / 2);
                    cp_async16(as + k * LDM + m, A + (int64_t)(k0 + k) * p.lda + i0 + m);
                }
            }
        } else {
#pragma unroll
        for (int r = 0; r < EPT; ++r) {
            const int idx = tid + r * kGemmThreads;
            int m, k, off;
            if (a_trans == 0) { k = idx % BK; m = idx / BK; off = m * kGemmLdk + k; }
            else { m = idx % BT; k = idx / BT; off = k * LDM + m; }
            const int gi = i0 + m, gk = k0 + k;
            const bool ok = gi < M && gk < kend;
            const double* src = ok ? (a_trans == 0 ? A + (int64_t)gi * p.lda + gk : A + (int64_t)gk * p.lda + gi) : A;
            cp_async8(as + off, src, ok);
        }
        }
        if (b_vec && kfull) {
#pragma unroll
            for (int r = 0; r < EPT / 2; ++r) {
                const int idx = tid + r * kGemmThreads;
                if (b_trans == 1) {
                    const int k = (idx % (BK / 2)) * 2, nn = idx / (BK / 2);
                    cp_async16(bs + nn * kGemmLdk + k, B + (int64_t)(j0 + nn) * p.ldb + k0 + k);
                } else {
                    const int nn = (idx % (BT / 2)) * 2, k = idx / (BT / 2);
                    cp_async16(bs + k * LDM + nn, B + (int64_t)(k0 + k) * p.ldb + j0 + nn);
                }
            }
            return;
        }
#pragma unroll
        for (int r = 0; r < EPT; ++r) {
            const int idx = tid + r * kGemmThreads;
            int n, k, off;
            if (b_trans == 1) { k = idx % BK; n = idx / BK; off = n * kGemmLdk + k; }
            else { n = idx % BT; k = idx / BT; off = k * LDM + n; }
            const int gj = j0 + n, gk = k0 + k;
            const bool ok = gj < N && gk < kend;
            const double* src = ok ? (b_trans == 1 ? B + (int64_t)gj * p.ldb + gk : B + (int64_t)gk * p.ldb + gj) : B;
            cp_async8(bs + off, src, ok);
        }
    };

    const int nkt = kbeg < kend ? (kend - kbeg + BK - 1) / BK : 0;
    // element (m, k) of the A tile and (k, n) of the B tile, in doubles
    const int a_sm = a_trans == 0 ? kGemmLdk : 1, a_sk = a_trans == 0 ? 1 : LDM;
    const int b_sn = b_trans == 1 ? kGemmLdk : 1, b_sk = b_trans == 1 ? 1 : LDM;
    const int a_lane = (wm0 + lq) * a_sm + lr * a_sk;
    const int b_lane = (wn0 + lq) * b_sn + lr * b_sk;

    for (int s = 0; s < kGemmStages - 1; ++s) {
        if (s < nkt) load_stage(s, kbeg + s * BK);
        cp_async_commit();
    }
    for (int kt = 0; kt < nkt; ++kt) {
        cp_async_wait<kGemmStages - 2>();
        __syncthreads();
        if (p.sym_double && kbeg + kt * BK == j0) {
#pragma unroll
            for (int a = 0; a < FM; ++a)
#pragma unroll
                for (int b = 0; b < FN; ++b) { acc[a][b][0] *= 2.0; acc[a][b][1] *= 2.0; }
        }
        if (kt + kGemmStages - 1 < nkt) load_stage((kt + kGemmStages - 1) % kGemmStages, kbeg + (kt + kGemmStages - 1) * BK);
        cp_async_commit();
        const double* as = smem + (size_t)(kt % kGemmStages) * 2 * TILE;
        const double* bs = as + TILE;
#pragma unroll
        for (int kk = 0; kk < BK; kk += 4) {
            double af[FM], bf[FN];
#pragma unroll
            for (int a = 0; a < FM; ++a) af[a] = as[a_lane + a * 8 * a_sm + kk * a_sk];
#pragma unroll
            for (int b = 0; b < FN; ++b) bf[b] = bs[b_lane + b * 8 * b_sn + kk * b_sk];
#pragma unroll
            for (int a = 0; a < FM; ++a)
#pragma unroll
                for (int b = 0; b < FN; ++b) dmma_884(acc[a][b][0], acc[a][b][1], af[a], bf[b]);
        }
    }
    cp_async_wait<0>();

    if (p.partials) {
        const double wgt = double_at_end ? 2.0 : 1.0;
        double s = 0.0;
#pragma unroll
        for (int a = 0; a < FM; ++a) {
            const int gi = i0 + wm0 + a * 8 + lq;
#pragma unroll
            for (int b = 0; b < FN; ++b)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int gj = j0 + wn0 + b * 8 + 2 * lr + e;
                    if (gi < M && gj < N) s = fma(acc[a][b][e], p.D[(int64_t)gi * p.ldd + gj], s);
                }
        }
        __syncthreads();
        double* red = smem;
        red[tid] = s;
        __syncthreads();
        for (int w = kGemmThreads / 2; w > 0; w >>= 1) {
            if (tid < w) red[tid] += red[tid + w];
            __syncthreads();
        }
        if (tid == 0)
            p.partials[((int64_t)zp * nby + by) * nbx + bx] = wgt * red[0];
        __syncthreads();
        return;
    }

    const bool do_mirror = p.mirror && (i0 != j0);
#pragma unroll
    for (int a = 0; a < FM; ++a) {
        const int gi = i0 + wm0 + a * 8 + lq;
        if (gi >= M) continue;
#pragma unroll
        for (int b = 0; b < FN; ++b)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int gj = j0 + wn0 + b * 8 + 2 * lr + e;
                if (gj >= N) continue;
                double v = p.alpha * acc[a][b][e];
                if (p.beta != 0.0) v = fma(p.beta, C[(int64_t)gi * p.ldc + gj], v);
                C[(int64_t)gi * p.ldc + gj] = v;
                if (do_mirror) C[(int64_t)gj * p.ldc + gi] = v;
            }
    }
}

// With sym_double the grid has half as many column tiles: CTA x handles column tiles x and nbx - 1 - x, whose k ranges
// (64 (x + 1) and 64 (nbx - x)) add up to the same length for every CTA.
template <int BT>
__global__ void __launch_bounds__(kGemmThreads, BT == 64 ? 2 : 1) dgemm_kernel(GemmParams p) {
    if (p.sym_double) {
        const int nbx = (p.N + BT - 1) / BT;
        const int bx = blockIdx.x, bx2 = nbx - 1 - bx;
        dgemm_tile<BT>(p, bx, blockIdx.y, blockIdx.z, nbx, gridDim.y);
        if (bx2 > bx) {
            __syncthreads();
            dgemm_tile<BT>(p, bx2, blockIdx.y, blockIdx.z, nbx, gridDim.y);
        }
        return;
    }
    dgemm_tile<BT>(p, blockIdx.x, blockIdx.y, blockIdx.z, gridDim.x, gridDim.y);
}

inline GemmParams gemm_defaults() {
    GemmParams p{};
    p.alpha = 1.0;
    p.beta = 0.0;
    return p;
}

// Launches with 128x128 tiles when that still fills the GPU, else 64x64.  Also reports the grid used.
inline int launch_dgemm(int kernel_id, const GemmParams& p, int batches, cudaStream_t stream, int force_bt = 0,
                        dim3* grid_out = nullptr) {
    DeviceState* dev = nullptr;
    int dst = current_device_state(&dev);
    if (dst) return dst;
    dst = ensure_smem_attr(dev, SA_DGEMM, [] {
        cudaError_t e = cudaFuncSetAttribute(dgemm_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)gemm_smem_bytes<128>());
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(dgemm_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)gemm_smem_bytes<64>());
        return e;
    });
    if (dst) return dst;
    if (p.M <= 0 || p.N <= 0 || batches <= 0) return PTQ_OK;
    int bt = force_bt;
    if (bt == 0) {
        const long tiles128 = (long)cdiv(p.M, 128) * cdiv(p.N, 128) * batches / (p.upper_only ? 2 : 1);
        bt = tiles128 >= 2 * dev->sms ? 128 : 64;
    }
    dim3 grid(cdiv(p.N, bt), cdiv(p.M, bt), p.ksplit > 1 ? p.ksplit : batches);
    if (grid_out) *grid_out = grid;          // the tile grid (what the partials are indexed by)
    if (p.sym_double) grid.x = (grid.x + 1) / 2;
    Launch scope(kernel_id, stream);
    if (bt == 128)
        dgemm_kernel<128><<<grid, kGemmThreads, gemm_smem_bytes<128>(), stream>>>(p);
    else
        dgemm_kernel<64><<<grid, kGemmThreads, gemm_smem_bytes<64>(), stream>>>(p);
    return launch_status();
}

}  // namespace ptq
