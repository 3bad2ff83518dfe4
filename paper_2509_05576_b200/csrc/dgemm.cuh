// Float64 GEMM tile kernel used by every float64 stage: the Cholesky trailing updates, the triangular
// inverse, Hinv = V V^T, the deferred Eq.-11 update of W, the float64 cross-check Gram and the loss
// 1/2 tr(dW H dW^T).  One kernel, parameterised by operand layout and by the triangular structure it
// may exploit.  All sums run over k in ascending order inside a tile, so results are deterministic.
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
};

constexpr int kGemmBK = 16;
constexpr int kGemmThreads = 256;

template <int BT>
constexpr size_t gemm_smem_bytes() { return size_t(2) * 2 * kGemmBK * (BT + 2) * sizeof(double); }

// BT x BT output tile, 256 threads, each thread owns (BT/16) x (BT/16) outputs as 2-wide groups spaced 32 apart.
template <int BT>
__global__ void __launch_bounds__(kGemmThreads) dgemm_kernel(GemmParams p) {
    constexpr int BK = kGemmBK;
    constexpr int LD = BT + 2;
    constexpr int T = BT / 16;        // outputs per thread per dimension
    constexpr int G = T / 2;          // 2-wide groups per dimension
    constexpr int EPT = BT * BK / kGemmThreads;  // elements each thread stages per operand tile
    extern __shared__ __align__(16) double smem[];
    double* As = smem;                    // [2][BK][LD]
    double* Bs = smem + 2 * BK * LD;      // [2][BK][LD]

    const int z = blockIdx.z;
    int N = p.N, K = p.K;
    if (p.ragN_step > 0) {
        int lim = p.ragN_lim - z * p.ragN_step;
        if (lim < N) N = lim;
        if (N <= 0) return;
    }
    if (p.k_is_n) K = N;
    const int M = p.M;
    const int i0 = blockIdx.y * BT, j0 = blockIdx.x * BT;
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

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;

    double acc[T][T];
#pragma unroll
    for (int a = 0; a < T; ++a)
#pragma unroll
        for (int b = 0; b < T; ++b) acc[a][b] = 0.0;

    double ra[EPT], rb[EPT];

    auto load_tiles = [&](int k0) {
#pragma unroll
        for (int r = 0; r < EPT; ++r) {
            int i, k;
            if (p.a_trans == 0) { k = tid & 15; i = (tid >> 4) + 16 * r; }
            else { i = tid % BT; k = tid / BT + (kGemmThreads / BT) * r; }
            const int gi = i0 + i, gk = k0 + k;
            double v = 0.0;
            if (gi < M && gk < kend)
                v = p.a_trans == 0 ? A[(int64_t)gi * p.lda + gk] : A[(int64_t)gk * p.lda + gi];
            ra[r] = v;
        }
#pragma unroll
        for (int r = 0; r < EPT; ++r) {
            int j, k;
            if (p.b_trans == 1) { k = tid & 15; j = (tid >> 4) + 16 * r; }
            else { j = tid % BT; k = tid / BT + (kGemmThreads / BT) * r; }
            const int gj = j0 + j, gk = k0 + k;
            double v = 0.0;
            if (gj < N && gk < kend)
                v = p.b_trans == 1 ? B[(int64_t)gj * p.ldb + gk] : B[(int64_t)gk * p.ldb + gj];
            rb[r] = v;
        }
    };
    auto store_tiles = [&](int buf) {
        double* as = As + buf * BK * LD;
        double* bs = Bs + buf * BK * LD;
#pragma unroll
        for (int r = 0; r < EPT; ++r) {
            int i, k;
            if (p.a_trans == 0) { k = tid & 15; i = (tid >> 4) + 16 * r; }
            else { i = tid % BT; k = tid / BT + (kGemmThreads / BT) * r; }
            as[k * LD + i] = ra[r];
        }
#pragma unroll
        for (int r = 0; r < EPT; ++r) {
            int j, k;
            if (p.b_trans == 1) { k = tid & 15; j = (tid >> 4) + 16 * r; }
            else { j = tid % BT; k = tid / BT + (kGemmThreads / BT) * r; }
            bs[k * LD + j] = rb[r];
        }
    };

    if (kbeg < kend) {
        load_tiles(kbeg);
        store_tiles(0);
        __syncthreads();
        int buf = 0;
        for (int k0 = kbeg; k0 < kend; k0 += BK) {
            const bool more = k0 + BK < kend;
            if (more) load_tiles(k0 + BK);
            const double* as = As + buf * BK * LD;
            const double* bs = Bs + buf * BK * LD;
#pragma unroll
            for (int k = 0; k < BK; ++k) {
                double av[T], bv[T];
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const double2 a2 = *reinterpret_cast<const double2*>(as + k * LD + g * 32 + ty * 2);
                    const double2 b2 = *reinterpret_cast<const double2*>(bs + k * LD + g * 32 + tx * 2);
                    av[2 * g] = a2.x; av[2 * g + 1] = a2.y;
                    bv[2 * g] = b2.x; bv[2 * g + 1] = b2.y;
                }
#pragma unroll
                for (int a = 0; a < T; ++a)
#pragma unroll
                    for (int b = 0; b < T; ++b) acc[a][b] = fma(av[a], bv[b], acc[a][b]);
            }
            if (more) store_tiles(buf ^ 1);
            __syncthreads();
            buf ^= 1;
        }
    }

    if (p.partials) {
        double s = 0.0;
#pragma unroll
        for (int a = 0; a < T; ++a) {
            const int gi = i0 + (a >> 1) * 32 + ty * 2 + (a & 1);
#pragma unroll
            for (int b = 0; b < T; ++b) {
                const int gj = j0 + (b >> 1) * 32 + tx * 2 + (b & 1);
                if (gi < M && gj < N) s = fma(acc[a][b], p.D[(int64_t)gi * p.ldd + gj], s);
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
            p.partials[((int64_t)z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x] = red[0];
        return;
    }

    const bool do_mirror = p.mirror && (i0 != j0);
#pragma unroll
    for (int a = 0; a < T; ++a) {
        const int gi = i0 + (a >> 1) * 32 + ty * 2 + (a & 1);
        if (gi >= M) continue;
#pragma unroll
        for (int b = 0; b < T; ++b) {
            const int gj = j0 + (b >> 1) * 32 + tx * 2 + (b & 1);
            if (gj >= N) continue;
            double v = p.alpha * acc[a][b];
            if (p.beta != 0.0) v = fma(p.beta, C[(int64_t)gi * p.ldc + gj], v);
            C[(int64_t)gi * p.ldc + gj] = v;
            if (do_mirror) C[(int64_t)gj * p.ldc + gi] = v;
        }
    }
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
    static bool attr_done = false;
    if (!attr_done) {
        cudaFuncSetAttribute(dgemm_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)gemm_smem_bytes<128>());
        cudaFuncSetAttribute(dgemm_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)gemm_smem_bytes<64>());
        attr_done = true;
    }
    if (p.M <= 0 || p.N <= 0 || batches <= 0) return PTQ_OK;
    int bt = force_bt;
    if (bt == 0) {
        const long tiles128 = (long)cdiv(p.M, 128) * cdiv(p.N, 128) * batches / (p.upper_only ? 2 : 1);
        bt = tiles128 >= 2 * 148 ? 128 : 64;
    }
    dim3 grid(cdiv(p.N, bt), cdiv(p.M, bt), batches);
    if (grid_out) *grid_out = grid;
    Launch scope(kernel_id, stream);
    if (bt == 128)
        dgemm_kernel<128><<<grid, kGemmThreads, gemm_smem_bytes<128>(), stream>>>(p);
    else
        dgemm_kernel<64><<<grid, kGemmThreads, gemm_smem_bytes<64>(), stream>>>(p);
    return launch_status();
}

}  // namespace ptq
