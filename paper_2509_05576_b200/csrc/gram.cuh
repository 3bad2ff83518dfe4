// H += 2 X X^T on the 5th-generation tensor cores, to float64 accuracy (Sec. 3: the Hessian of Eq. 2).
//
// The column order and the rounding decisions of the method are sensitive to errors in H far below
// float32 resolution, so the product is formed from error-free integer slices:
//   every row x_i of X is scaled by a power of two 2^sh_i so that |x| 2^sh_i < 2^46, rounded to an integer v
//   (exact for float32 data within 2^-46 of the row maximum) and written as six balanced base-256 digits,
//       v = sum_{s=0..5} d_s 256^(5-s),  d_s in [-128, 127]  (int8 "slices", most significant first).
//   Then  sum_k v_ik v_jk = sum_{a,b} 256^(10-a-b) (D_a D_b^T)_ij, and each D_a D_b^T is an exact int8 x int8 -> int32
//   tensor-core product.  Slice pairs with a + b = t share the weight 256^(10-t), so one int32 accumulator G_t per
//   group t is enough; groups t <= 5 are kept (21 pair products), the dropped ones weigh 2^-48 and less.
//
// Kernel: one 128 x 64 output tile per CTA iteration (upper triangle only, mirrored on store).  A TMA producer warp
// streams 64-wide K blocks of all six slices of the 128 "row" columns and of the 64 "column" columns
// (SWIZZLE_64B, 3 stages of 72 KB); one thread issues the 42 tcgen05.mma.kind::i8 instructions of a stage into six
// TMEM accumulators (6 x 64 columns); four epilogue warps read the accumulators back with tcgen05.ld, combine the
// groups exactly in int64, hand TMEM back (the next tile's products then overlap the rest of the epilogue), scale by
// 2^(41 - sh_i - sh_j) and add into H.
// Every wait on an mbarrier is bounded; when one expires the CTA records PTQ_ERR_TIMEOUT, drains and returns.
#pragma once
#include "common.cuh"

namespace ptq {

constexpr int kSlices = 6;
constexpr int kGroups = 6;                 // groups t = a + b = 0..5
constexpr int kGramTM = 128;               // tile rows
constexpr int kGramTN = 64;                // tile columns
constexpr int kGramKB = 64;                // K block (int8 elements = bytes)
constexpr int kGramStages = 3;
constexpr int kGramABytes = kGramTM * kGramKB;                    // 8 KB per slice
constexpr int kGramBBytes = kGramTN * kGramKB;                    // 4 KB per slice
constexpr int kGramStageBytes = kSlices * (kGramABytes + kGramBBytes);   // 72 KB
constexpr int kGramSmemBytes = kGramStages * kGramStageBytes + 1024 /*align*/ + 256 /*barriers*/;
constexpr int kGramThreads = 192;          // warp 0: TMA, warp 1: MMA + TMEM, warps 2..5: epilogue
constexpr int kGramMaxChunk = 16384;       // calibration columns per launch: 6 * 2^14 * 16384 < 2^31
constexpr int kShiftTarget = 46;

constexpr int kGramMaxSplit = 16;          // slices of the K range per tile
constexpr int kGramMaxSplitTiles = 128;    // tiles of one launch whose K range may be cut across CTAs
constexpr size_t kGramTileAccWords = 2 * (size_t)kGramTM * kGramTN;   // int64 words per such tile (high and low sums)

inline int gram_num_tiles(int cols) {
    const int nbi = cdiv(cols, kGramTM), nbj = cdiv(cols, kGramTN);
    int t = 0;
    for (int b = 0; b < nbi; ++b) t += (nbj - 2 * b) > 0 ? (nbj - 2 * b) : 0;
    return t;
}

inline size_t gram_workspace_bytes(int cols, int n) {
    const size_t cols_pad = (size_t)cdiv(cols, 128) * 128;
    const int chunk = n < kGramMaxChunk ? n : kGramMaxChunk;
    const size_t n_pad = (size_t)cdiv(chunk, 128) * 128;
    size_t total = align_up(kSlices * cols_pad * n_pad) + align_up(cols_pad * sizeof(int32_t));
    const int tiles = gram_num_tiles(cols);
    total += align_up((size_t)(tiles < kGramMaxSplitTiles ? tiles : kGramMaxSplitTiles) * kGramTileAccWords *
                      sizeof(long long));
    return total;
}

// ------------------------------------------------------------------------------------------------------------
// Where the rows of X come from.  Either a plain [cols x n] matrix, or the input of a convolution whose unfolded
// patches ARE the columns of X (Sec. 3: for a convolutional layer d_col is the number of weights of one filter, so row
// (c, ki, kj) of X holds, for every image b and output position (oy, ox), the input value that weight multiplies):
//     X[(c kh + ki) kw + kj][(b OH + oy) OW + ox] = act[b][c][oy stride + ki - pad][ox stride + kj - pad]   (0 outside)
// The patches are never materialised in float32: the slicing pre-pass reads the activations in place.
// ------------------------------------------------------------------------------------------------------------
struct GramSource {
    const float* base;      // X, or the activations [batch][channels][height][width]
    int64_t ldx;            // matrix: row stride
    int conv;               // 0: matrix, 1: convolution input
    int channels, height, width, kh, kw, stride, pad, oh, ow;
    int col0;               // first calibration column of this launch
};

// ------------------------------------------------------------------------------------------------------------
// Slicing pre-pass: one CTA per (padded) row.
// ------------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gram_split_conv_kernel(GramSource src, int cols, int n, int cols_pad, int n_pad,
                                                               int8_t* __restrict__ Q, int32_t* __restrict__ shifts,
                                                               int32_t* status);

__device__ __forceinline__ void gram_pack4(const long long (&v)[4], uint32_t (&packed)[kSlices]) {
#pragma unroll
    for (int s = 0; s < kSlices; ++s) packed[s] = 0u;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        long long t = v[u];
#pragma unroll
        for (int s = kSlices - 1; s >= 0; --s) {          // least significant digit first
            const long long d = ((t + 128) & 255) - 128;  // balanced digit in [-128, 127]
            t = (t - d) >> 8;
            packed[s] |= ((uint32_t)(d & 255)) << (8 * u);
        }
    }
}

__global__ void __launch_bounds__(256) gram_split_kernel(const float* __restrict__ X, int cols, int n, int64_t ldx,
                                                          int cols_pad, int n_pad, int vec_ok,
                                                          int8_t* __restrict__ Q, int32_t* __restrict__ shifts,
                                                          int32_t* status) {
    __shared__ float smax[256];
    __shared__ int sbad;
    const int row = blockIdx.x;
    const size_t plane = (size_t)cols_pad * n_pad;
    int8_t* q0 = Q + (size_t)row * n_pad;
    if (row >= cols) {   // padding rows: zeros
        for (int k = threadIdx.x * 4; k < n_pad; k += 1024)
#pragma unroll
            for (int s = 0; s < kSlices; ++s) *reinterpret_cast<uint32_t*>(q0 + s * plane + k) = 0u;
        if (threadIdx.x == 0) shifts[row] = 0;
        return;
    }
    if (threadIdx.x == 0) sbad = 0;
    __syncthreads();
    const float* x = X + (int64_t)row * ldx;
    float m = 0.f;
    bool bad = false;
    for (int k = threadIdx.x * 4; k < n; k += 1024) {
        if (vec_ok && k + 3 < n) {
            const float4 v = *reinterpret_cast<const float4*>(x + k);
            bad |= !isfinite(v.x) | !isfinite(v.y) | !isfinite(v.z) | !isfinite(v.w);
            m = fmaxf(m, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
        } else {
            for (int kk = k; kk < n; ++kk) { bad |= !isfinite(x[kk]); m = fmaxf(m, fabsf(x[kk])); }
        }
    }
    if (bad) sbad = 1;
    smax[threadIdx.x] = m;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (threadIdx.x < w) smax[threadIdx.x] = fmaxf(smax[threadIdx.x], smax[threadIdx.x + w]);
        __syncthreads();
    }
    const float rowmax = smax[0];
    const bool rowbad = sbad != 0;
    if (rowbad && threadIdx.x == 0) report(status, PTQ_ERR_NONFINITE, row);
    int sh = 0;
    if (rowmax > 0.f && !rowbad) sh = kShiftTarget - (ilogbf(rowmax) + 1);   // |x| 2^sh < 2^46
    if (threadIdx.x == 0) shifts[row] = sh;
    for (int k = threadIdx.x * 4; k < n_pad; k += 1024) {
        long long v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int kk = k + u;
            const float xv = (kk < n && !rowbad) ? x[kk] : 0.f;
            v[u] = __double2ll_rn(scalbn((double)xv, sh));
        }
        uint32_t packed[kSlices];
        gram_pack4(v, packed);
#pragma unroll
        for (int s = 0; s < kSlices; ++s) *reinterpret_cast<uint32_t*>(q0 + s * plane + k) = packed[s];
    }
}

// The same pre-pass reading the input of a convolution in place (see GramSource).  Thread t walks the calibration
// columns 4 t .. 4 t + 3, 4 t + 1024 .., keeping (image, output row, output column) up to date by carries.
struct ConvCursor {
    int b, oy, ox;
    __device__ __forceinline__ void set(const GramSource& s, int col) {
        const int per = s.oh * s.ow;
        b = col / per;
        const int r = col - b * per;
        oy = r / s.ow;
        ox = r - oy * s.ow;
    }
    __device__ __forceinline__ void next(const GramSource& s) {
        if (++ox == s.ow) { ox = 0; if (++oy == s.oh) { oy = 0; ++b; } }
    }
};
__device__ __forceinline__ float conv_fetch(const GramSource& s, const float* __restrict__ plane0, const ConvCursor& c,
                                            int ki, int kj) {
    const int iy = c.oy * s.stride + ki - s.pad, ix = c.ox * s.stride + kj - s.pad;
    if ((unsigned)iy >= (unsigned)s.height || (unsigned)ix >= (unsigned)s.width) return 0.f;
    return plane0[((int64_t)c.b * s.channels * s.height + iy) * s.width + ix];
}

__global__ void __launch_bounds__(256) gram_split_conv_kernel(GramSource src, int cols, int n, int cols_pad, int n_pad,
                                                               int8_t* __restrict__ Q, int32_t* __restrict__ shifts,
                                                               int32_t* status) {
    __shared__ float smax[256];
    __shared__ int sbad;
    const int row = blockIdx.x;
    const size_t plane = (size_t)cols_pad * n_pad;
    int8_t* q0 = Q + (size_t)row * n_pad;
    if (row >= cols) {   // padding rows: zeros
        for (int k = threadIdx.x * 4; k < n_pad; k += 1024)
#pragma unroll
            for (int s = 0; s < kSlices; ++s) *reinterpret_cast<uint32_t*>(q0 + s * plane + k) = 0u;
        if (threadIdx.x == 0) shifts[row] = 0;
        return;
    }
    if (threadIdx.x == 0) sbad = 0;
    __syncthreads();
    const int kk2 = src.kh * src.kw;
    const int ch = row / kk2, rem = row - ch * kk2;
    const int ki = rem / src.kw, kj = rem - ki * src.kw;
    const float* plane0 = src.base + (int64_t)ch * src.height * src.width;     // channel ch of image 0
    float m = 0.f;
    bool bad = false;
    for (int k = threadIdx.x * 4; k < n; k += 1024) {
        ConvCursor cur;
        cur.set(src, src.col0 + k);
        for (int u = 0; u < 4 && k + u < n; ++u) {
            const float xv = conv_fetch(src, plane0, cur, ki, kj);
            bad |= !isfinite(xv);
            m = fmaxf(m, fabsf(xv));
            cur.next(src);
        }
    }
    if (bad) sbad = 1;
    smax[threadIdx.x] = m;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if (threadIdx.x < w) smax[threadIdx.x] = fmaxf(smax[threadIdx.x], smax[threadIdx.x + w]);
        __syncthreads();
    }
    const float rowmax = smax[0];
    const bool rowbad = sbad != 0;
    if (rowbad && threadIdx.x == 0) report(status, PTQ_ERR_NONFINITE, row);
    int sh = 0;
    if (rowmax > 0.f && !rowbad) sh = kShiftTarget - (ilogbf(rowmax) + 1);   // |x| 2^sh < 2^46
    if (threadIdx.x == 0) shifts[row] = sh;
    for (int k = threadIdx.x * 4; k < n_pad; k += 1024) {
        long long v[4];
        ConvCursor cur;
        cur.set(src, src.col0 + k);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float xv = (k + u < n && !rowbad) ? conv_fetch(src, plane0, cur, ki, kj) : 0.f;
            v[u] = __double2ll_rn(scalbn((double)xv, sh));
            cur.next(src);
        }
        uint32_t packed[kSlices];
        gram_pack4(v, packed);
#pragma unroll
        for (int s = 0; s < kSlices; ++s) *reinterpret_cast<uint32_t*>(q0 + s * plane + k) = packed[s];
    }
}

// ------------------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------------------
// Bounded wait: gives up after about a second of polling or as soon as another thread of the CTA gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const long long t0 = clock64();
    uint32_t it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 255u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > 2000000000LL) { *abort_flag = 1; return false; }
        }
    }
    return true;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tmap, int c0, int c1, int c2,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(tmap), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}\n"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 64-byte rows, SWIZZLE_64B; 8-row groups are 512 bytes apart.
__device__ __forceinline__ uint64_t make_desc_sw64(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);        // start address / 16
    d |= (uint64_t)1 << 16;                            // leading byte offset / 16 (not used by swizzled K-major)
    d |= (uint64_t)(512 >> 4) << 32;                   // stride byte offset / 16
    d |= (uint64_t)1 << 46;                            // descriptor version of this architecture
    d |= (uint64_t)4 << 61;                            // SWIZZLE_64B
    return d;
}

// The same descriptor as two 32-bit words; the address field (bits 0..13, shared-memory address / 16) is added to the
// low word at run time: all tiles lie below 256 KB, so the sum never leaves the field.
constexpr uint32_t kDescLo = 1u << 16;
constexpr uint32_t kDescHi = (uint32_t)(512 >> 4) | (1u << 14) | (4u << 29);
__device__ __forceinline__ void tc_mma_i8_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi,
                                               uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, {%6, %6, %6, %6}, p;\n\t}\n"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}

// Instruction descriptor: int8 x int8 -> int32, both operands K-major, M = 128, N = 64.
constexpr uint32_t kGramIdesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kGramTN >> 3) << 17) |
                                ((uint32_t)(kGramTM >> 4) << 24);

// Tile t of the enumeration: row block bi (128 rows), column block bj (64 columns) with 64*bj + 63 >= 128*bi.
__device__ __forceinline__ void gram_tile_coords(int tile, int nbj, int& bi, int& bj) {
    int b = 0, rem = tile;
    for (;;) {
        const int cnt = nbj - 2 * b;    // column blocks 2b .. nbj-1
        if (rem < cnt) break;
        rem -= cnt;
        ++b;
    }
    bi = b;
    bj = 2 * b + rem;
}

__global__ void __launch_bounds__(kGramThreads, 1)
gram_i8_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
               double* __restrict__ H, int cols, int n_pad,
               const int32_t* __restrict__ shifts, int num_tiles, int nbj, int32_t* status, int n_full, int ksplit,
               unsigned long long* __restrict__ iacc) {
    extern __shared__ unsigned char gram_smem_raw[];
    const uint32_t raw = smem_u32(gram_smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* base_ptr = gram_smem_raw + (base - raw);
    // barriers live after the stages
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + kGramStages * kGramStageBytes);
    const uint32_t bar0 = base + kGramStages * kGramStageBytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kGramStages + s); };
    const uint32_t acc_full = bar0 + 8u * (2 * kGramStages);
    const uint32_t acc_empty = bar0 + 8u * (2 * kGramStages + 1);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kGramStages + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nkb = n_pad / kGramKB;
    // Work items: the first n_full tiles whole, then the remaining tiles cut into ksplit slices of the K range each
    // (a last, partly filled wave of tiles, or all tiles of a narrow matrix, spread over every SM this way).
    const int klen = (nkb + ksplit - 1) / ksplit;
    const int num_items = n_full + (num_tiles - n_full) * ksplit;
    auto item_tile = [&](int item) { return item < n_full ? item : n_full + (item - n_full) / ksplit; };
    auto item_kb0 = [&](int item) { return item < n_full ? 0 : ((item - n_full) % ksplit) * klen; };
    auto item_kb1 = [&](int item) {
        if (item < n_full) return nkb;
        const int e = item_kb0(item) + klen;
        return e < nkb ? e : nkb;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGramStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
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
            int armed[kGramStages];
#pragma unroll
            for (int s = 0; s < kGramStages; ++s) armed[s] = -1;
            bool ok = true;
            for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
                int bi, bj;
                gram_tile_coords(item_tile(item), nbj, bi, bj);
                const int kb0 = item_kb0(item), kb1 = item_kb1(item);
                for (int kb = kb0; kb < kb1 && ok; ++kb) {
                    ok = mbar_wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag);
                    if (!ok) break;
                    const uint32_t sbase = base + stage * kGramStageBytes;
                    mbar_arrive_expect_tx(full_bar(stage), kGramStageBytes);
                    armed[stage] = (int)phase;
#pragma unroll
                    for (int s = 0; s < kSlices; ++s) {
                        tma_load_3d(sbase + s * kGramABytes, &tmapA, kb * kGramKB, bi * kGramTM, s, full_bar(stage));
                        tma_load_3d(sbase + kSlices * kGramABytes + s * kGramBBytes, &tmapB, kb * kGramKB,
                                    bj * kGramTN, s, full_bar(stage));
                    }
                    if (++stage == kGramStages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // drain: wait (bounded) until the copies already issued have landed
                for (int s = 0; s < kGramStages; ++s)
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
            for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
                ok = mbar_wait_bounded(acc_empty, acc_phase ^ 1u, abort_flag);   // epilogue has drained TMEM
                if (!ok) break;
                tc_fence_after();
                const int kb0 = item_kb0(item), kb1 = item_kb1(item);
                for (int kb = kb0; kb < kb1 && ok; ++kb) {
                    ok = mbar_wait_bounded(full_bar(stage), phase, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    // Descriptors: A and B tiles share the high word; the low word is the stage's address field plus a
                    // compile-time offset per slice and per 32-byte K step, so each MMA costs two integer adds.
                    const uint32_t sb = kDescLo + ((base + stage * kGramStageBytes) >> 4);
                    const uint32_t first = kb > kb0 ? 1u : 0u;    // the first product of a group overwrites
#pragma unroll
                    for (int t = 0; t < kGroups; ++t) {
#pragma unroll
                        for (int a = 0; a <= t; ++a) {
                            const int b = t - a;
#pragma unroll
                            for (int ks = 0; ks < kGramKB / 32; ++ks) {
                                const uint32_t alo = sb + (uint32_t)((a * kGramABytes) >> 4) + (uint32_t)(ks * 2);
                                const uint32_t blo = sb + (uint32_t)((kSlices * kGramABytes + b * kGramBBytes) >> 4) +
                                                     (uint32_t)(ks * 2);
                                tc_mma_i8_lohi(tmem_base + t * kGramTN, alo, blo, kDescHi, kGramIdesc,
                                               (a > 0 || ks > 0) ? 1u : first);
                            }
                        }
                    }
                    tc_commit(empty_bar(stage));     // the stage may be refilled once these MMAs have read it
                    if (++stage == kGramStages) { stage = 0; phase ^= 1u; }
                }
                if (ok) tc_commit(acc_full);         // accumulators complete
                acc_phase ^= 1u;
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (warps 2..5)
        const int quarter = warp & 3;                 // TMEM lanes this warp may read
        const int r_in_tile = quarter * 32 + lane;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
            int bi, bj;
            const int tile = item_tile(item);
            const bool sliced = item >= n_full && ksplit > 1;
            gram_tile_coords(tile, nbj, bi, bj);
            ok = mbar_wait_bounded(acc_full, acc_phase, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const int row = bi * kGramTM + r_in_tile;
            const int sh_i = row < cols ? shifts[row] : 0;
            // 1. drain the accumulators into registers: v = G0 2^40 + G1 2^32 + ... + G5, combined exactly in int64 and
            //    rounded once to float64; then TMEM is handed back, so that the next tile's products run under step 2
            double v[kGramTN];
#pragma unroll
            for (int ch = 0; ch < kGramTN / 16; ++ch) {
                long long lo[16], hi[16];
                uint32_t r[16];
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + ch * 16;
                // groups 5, 4, 3 -> lo = G5 + 2^8 G4 + 2^16 G3 ; groups 2, 1, 0 -> hi = G2 + 2^8 G1 + 2^16 G0
                tc_ld16(taddr + 5 * kGramTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) lo[c] = (long long)(int)r[c];
                tc_ld16(taddr + 4 * kGramTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) lo[c] += (long long)(int)r[c] << 8;
                tc_ld16(taddr + 3 * kGramTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) lo[c] += (long long)(int)r[c] << 16;
                tc_ld16(taddr + 2 * kGramTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) hi[c] = (long long)(int)r[c];
                tc_ld16(taddr + 1 * kGramTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) hi[c] += (long long)(int)r[c] << 8;
                tc_ld16(taddr + 0 * kGramTN, r); tc_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c) hi[c] += (long long)(int)r[c] << 16;
                if (sliced) {
                    // a slice of the K range: the exact integer sums go to the tile's workspace (integer atomics commute,
                    // so the total does not depend on the order of the slices); column-major, rows contiguous
                    unsigned long long* acc = iacc + (size_t)(tile - n_full) * kGramTileAccWords;
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const int idx = (ch * 16 + c) * kGramTM + r_in_tile;
                        atomicAdd(acc + idx, (unsigned long long)hi[c]);
                        atomicAdd(acc + kGramTM * kGramTN + idx, (unsigned long long)lo[c]);
                    }
                }
#pragma unroll
                for (int c = 0; c < 16; ++c) v[ch * 16 + c] = fma((double)hi[c], 16777216.0, (double)lo[c]);
            }
            tc_fence_before();
            mbar_arrive(acc_empty);
            acc_phase ^= 1u;
            // 2. H += v 2^(41 - sh_i - sh_j).  Tiles away from the diagonal also own the mirrored entries (j, i); since H
            //    is symmetric the old value is read there, where consecutive lanes (rows i) are contiguous.
            if (row < cols && !sliced) {
                const bool straddle = (bj * kGramTN < bi * kGramTM + kGramTM);
                const double fi = __longlong_as_double((long long)(1023 + 20 - sh_i) << 52);     // 2^(20 - sh_i)
#pragma unroll
                for (int c = 0; c < kGramTN; ++c) {
                    const int col = bj * kGramTN + c;
                    if (col < cols) {
                        const double fj = __longlong_as_double((long long)(1023 + 21 - shifts[col]) << 52);
                        const double add = (v[c] * fi) * fj;                // exact: powers of two, no under/overflow
                        if (straddle) {
                            // tiles that straddle the diagonal hold both (i, j) and (j, i): each writes itself only
                            H[(int64_t)row * cols + col] += add;
                        } else {
                            const double out = H[(int64_t)col * cols + row] + add;
                            H[(int64_t)col * cols + row] = out;
                            H[(int64_t)row * cols + col] = out;
                        }
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
    if (threadIdx.x == 0 && *abort_flag) report(status, PTQ_ERR_TIMEOUT, blockIdx.x);
}

// After a launch with sliced tiles: for each of them, H += (hi 2^24 + lo) 2^(41 - sh_i - sh_j) from the integer sums,
// rounded once and written exactly as the unsliced epilogue does (so the result is the same bit for bit).
// One CTA per sliced tile and group of 16 columns, one thread per row of the tile.
__global__ void __launch_bounds__(kGramTM) gram_finish_kernel(const unsigned long long* __restrict__ iacc,
                                                               double* __restrict__ H, int cols, int n_full, int nbj,
                                                               const int32_t* __restrict__ shifts) {
    const int tile = n_full + blockIdx.x;
    int bi, bj;
    gram_tile_coords(tile, nbj, bi, bj);
    const int row = bi * kGramTM + threadIdx.x;
    if (row >= cols) return;
    const unsigned long long* acc = iacc + (size_t)blockIdx.x * kGramTileAccWords;
    const bool straddle = (bj * kGramTN < bi * kGramTM + kGramTM);
    const double fi = __longlong_as_double((long long)(1023 + 20 - shifts[row]) << 52);
#pragma unroll 4
    for (int cc = 0; cc < 16; ++cc) {
        const int c = blockIdx.y * 16 + cc, col = bj * kGramTN + c;
        if (col >= cols) continue;
        const long long hi = (long long)acc[c * kGramTM + threadIdx.x];
        const long long lo = (long long)acc[kGramTM * kGramTN + c * kGramTM + threadIdx.x];
        const double v = fma((double)hi, 16777216.0, (double)lo);
        const double fj = __longlong_as_double((long long)(1023 + 21 - shifts[col]) << 52);
        const double add = (v * fi) * fj;
        if (straddle) {
            H[(int64_t)row * cols + col] += add;
        } else {
            const double out = H[(int64_t)col * cols + row] + add;
            H[(int64_t)col * cols + row] = out;
            H[(int64_t)row * cols + col] = out;
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------------------
inline int make_slice_map(CUtensorMap* m, int8_t* Q, int cols_pad, int n_pad, int box_rows) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return PTQ_ERR_CUDA;
    const cuuint64_t dims[3] = {(cuuint64_t)n_pad, (cuuint64_t)cols_pad, (cuuint64_t)kSlices};
    const cuuint64_t strides[2] = {(cuuint64_t)n_pad, (cuuint64_t)cols_pad * (cuuint64_t)n_pad};
    const cuuint32_t box[3] = {(cuuint32_t)kGramKB, (cuuint32_t)box_rows, 1u};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, Q, dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PTQ_OK : PTQ_ERR_CUDA;
}

inline int gram_accumulate(double* H, GramSource src, int cols, int n, void* ws, int32_t* status,
                           cudaStream_t stream) {
    DeviceState* dev = nullptr;
    int dst = current_device_state(&dev);
    if (dst) return dst;
    dst = ensure_smem_attr(dev, SA_GRAM, [] {
        return cudaFuncSetAttribute(gram_i8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGramSmemBytes);
    });
    if (dst) return dst;
    const int num_sms = dev->sms;
    const int cols_pad = cdiv(cols, 128) * 128;
    const int max_chunk = n < kGramMaxChunk ? n : kGramMaxChunk;
    const size_t n_pad_max = (size_t)cdiv(max_chunk, 128) * 128;
    Carver cv(ws);
    int8_t* Q = cv.take<int8_t>(kSlices * (size_t)cols_pad * n_pad_max);
    int32_t* shifts = cv.take<int32_t>(cols_pad);
    const int nbj = cdiv(cols, kGramTN);
    const int num_tiles = gram_num_tiles(cols);
    unsigned long long* iacc = cv.take<unsigned long long>(
        (size_t)(num_tiles < kGramMaxSplitTiles ? num_tiles : kGramMaxSplitTiles) * kGramTileAccWords);
    for (int c0 = 0; c0 < n; c0 += kGramMaxChunk) {
        const int nc = n - c0 < kGramMaxChunk ? n - c0 : kGramMaxChunk;
        const int n_pad = cdiv(nc, 128) * 128;
        {
            Launch l(K_GRAM_SPLIT, stream);
            if (src.conv) {
                src.col0 = c0;
                gram_split_conv_kernel<<<cols_pad, 256, 0, stream>>>(src, cols, nc, cols_pad, n_pad, Q, shifts, status);
            } else {
                const int vec_ok = (aligned16(src.base) && (src.ldx & 3) == 0) ? 1 : 0;
                gram_split_kernel<<<cols_pad, 256, 0, stream>>>(src.base + c0, cols, nc, src.ldx, cols_pad, n_pad, vec_ok,
                                                                Q, shifts, status);
            }
        }
        CUtensorMap mapA, mapB;
        int st = make_slice_map(&mapA, Q, cols_pad, n_pad, kGramTM);
        if (st) return st;
        st = make_slice_map(&mapB, Q, cols_pad, n_pad, kGramTN);
        if (st) return st;
        // The tiles of the last, partly filled wave (all tiles of a narrow matrix) are cut along K so that every SM
        // gets a work item of about the same length.
        const int nkb = n_pad / kGramKB;
        const int rem = num_tiles % num_sms;
        int n_full = num_tiles, ksplit = 1;
        if (rem > 0 && rem <= kGramMaxSplitTiles && 2 * rem <= num_sms) {
            ksplit = num_sms / rem;
            if (ksplit > kGramMaxSplit) ksplit = kGramMaxSplit;
            if (ksplit > nkb / 2) ksplit = nkb / 2 > 0 ? nkb / 2 : 1;
            ksplit = cdiv(nkb, cdiv(nkb, ksplit));          // no empty slice
            if (ksplit > 1) n_full = num_tiles - rem;
        }
        const int sliced = num_tiles - n_full;
        if (sliced > 0 &&
            cudaMemsetAsync(iacc, 0, (size_t)sliced * kGramTileAccWords * sizeof(unsigned long long), stream) != cudaSuccess)
            return PTQ_ERR_CUDA;
        const int items = n_full + sliced * ksplit;
        const int grid = items < num_sms ? items : num_sms;
        {
            Launch l(K_GRAM_I8, stream);
            gram_i8_kernel<<<grid, kGramThreads, kGramSmemBytes, stream>>>(mapA, mapB, H, cols, n_pad, shifts,
                                                                         num_tiles, nbj, status, n_full, ksplit, iacc);
        }
        if (sliced > 0) {
            Launch l(K_GRAM_FINISH, stream);
            gram_finish_kernel<<<dim3(sliced, kGramTN / 16), kGramTM, 0, stream>>>(iacc, H, cols, n_full, nbj, shifts);
        }
        if (cudaGetLastError() != cudaSuccess) return PTQ_ERR_CUDA;
    }
    return PTQ_OK;
}

}  // namespace ptq
