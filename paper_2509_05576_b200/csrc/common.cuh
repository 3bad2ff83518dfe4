// Shared host/device helpers of the quantizer library (status word, launch checks, workspace carving).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include <mutex>
#include <vector>

#include "../../include/ptq.h"

namespace ptq {

constexpr int kNB = 64;  // block size of the factorisations and of the column loop

// First error wins; later kernels keep running on whatever numbers they find (no traps, no faults).
__device__ __forceinline__ void report(int32_t* status, int code, int index, int aux = 0) {
    if (status && atomicCAS(status, 0, code) == 0) {
        status[1] = index;
        status[2] = aux;
    }
}

// ---------------------------------------------------------------------------------------------------------
// Shared-memory barriers and tensor-map (TMA) tile copies used by the tile pipelines.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

// Carves aligned pieces out of the caller's workspace.
struct Carver {
    char* base;
    size_t off = 0;
    explicit Carver(void* p) : base(static_cast<char*>(p)) {}
    template <typename T>
    T* take(size_t count) {
        T* p = reinterpret_cast<T*>(base + off);
        off = align_up(off + count * sizeof(T));
        return p;
    }
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? PTQ_OK : PTQ_ERR_CUDA; }

inline int cdiv(int a, int b) { return (a + b - 1) / b; }

// Bounded device-side waits give up after this many SM clock cycles (about two seconds).
constexpr long long kSpinLimitCycles = 4000000000LL;

// ---------------------------------------------------------------------------------------------------------
// Host-side state that belongs to a DEVICE, not to the process: the SM count that sizes the persistent grids, the
// cooperative-launch capability and which kernels already carry their dynamic shared-memory attribute there
// (cudaFuncSetAttribute is per device).  One table, one mutex; looked up with the caller's device current.
// ---------------------------------------------------------------------------------------------------------
constexpr int kMaxDevices = 64;
enum SmemAttrSlot { SA_CHOL = 0, SA_SWEEP, SA_GRAM, SA_DGEMM, SA_SMALL, SA_XGEMM, SA_COUNT };
struct DeviceState {
    int sms = 0;
    int coop = 0;
    int cta_limit = 0;            // > 0: the persistent cooperative kernels launch at most this many CTAs (ptq_set_cta_limit)
    bool attr[SA_COUNT] = {};
};
inline std::mutex& host_state_mutex() { static std::mutex mu; return mu; }
inline int current_device_state(DeviceState** out) {
    static DeviceState table[kMaxDevices];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PTQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(host_state_mutex());
    DeviceState& d = table[dev];
    if (d.sms == 0) {
        int sms = 0, coop = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return PTQ_ERR_CUDA;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess) return PTQ_ERR_CUDA;
        d.coop = coop;
        d.sms = sms;
    }
    *out = &d;
    return PTQ_OK;
}
// CTAs a persistent cooperative kernel may launch on this device: one per SM, or the caller's limit if that is lower.
inline int coop_cta_budget(const DeviceState* d) {
    std::lock_guard<std::mutex> lock(host_state_mutex());
    return (d->cta_limit > 0 && d->cta_limit < d->sms) ? d->cta_limit : d->sms;
}
// Runs `set` (the cudaFuncSetAttribute calls of one kernel family) once per device.
template <typename F>
inline int ensure_smem_attr(DeviceState* d, SmemAttrSlot slot, F set) {
    std::lock_guard<std::mutex> lock(host_state_mutex());
    if (!d->attr[slot]) {
        if (set() != cudaSuccess) { cudaGetLastError(); return PTQ_ERR_CUDA; }
        d->attr[slot] = true;
    }
    return PTQ_OK;
}

// ---------------------------------------------------------------------------------------------------------
// Launch accounting.  Every kernel launch of the library goes through a Launch scope: it always counts the
// launch, and, while profiling is enabled, brackets it with CUDA events on the launching stream so that the
// bench can read per-kernel device time live.  Profiling adds event records between kernels, so it is used on
// separate, untimed passes.
// ---------------------------------------------------------------------------------------------------------
enum KernelId {
    K_GRAM_SPLIT = 0, K_GRAM_I8, K_GRAM_FINISH, K_CONVERT_F64, K_DGEMM_GRAM, K_LAMBDA, K_DAMP_COPY, K_CHOL_COOP,
    K_DGEMM_LAUUM, K_EXTRACT_DIAG, K_MINMAX_GRID, K_SCORE_PARTIAL,
    K_SCORE_FINAL, K_RANK_SORT, K_PERM_CHECK, K_GATHER_SYM, K_GATHER_W, K_SWEEP_COOP, K_FINALIZE,
    K_DGEMM_LOSS, K_SUM_PARTIALS, K_SELFTEST, K_FP64_PROBE, K_DYN_AUX, K_DYN_GATHER,
    K_DGEMM_DYN, K_PER_ROW, K_DGEMM_EQ11, K_X_SLICE, K_X_GEMM, K_COUNT
};

inline const char* kernel_name(int id) {
    static const char* names[K_COUNT] = {
        "gram_split", "gram_i8_tcgen05", "gram_finish", "convert_f64", "dgemm_gram_f64", "lambda", "damp_copy", "chol_coop",
        "dgemm_lauum", "extract_diag",
        "minmax_grid", "score_partial", "score_final", "rank_sort", "perm_check", "gather_sym", "gather_w",
        "sweep_coop", "finalize", "dgemm_loss", "sum_partials", "selftest_wait", "fp64_probe", "dyn_aux", "dyn_gather",
        "dgemm_dyn", "per_row", "dgemm_eq11", "x_slice", "i8gemm_tcgen05"};
    return (id >= 0 && id < K_COUNT) ? names[id] : "unknown";
}

struct Profiler {
    bool on = false;
    long long launches[K_COUNT] = {};
    struct Rec { int id; cudaEvent_t a, b; };
    std::vector<Rec> recs;
    std::vector<cudaEvent_t> pool;
    cudaEvent_t get() {
        if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
    void clear() {
        for (auto& r : recs) { pool.push_back(r.a); pool.push_back(r.b); }
        recs.clear();
    }
};
inline Profiler& profiler() { static Profiler p; return p; }

inline std::mutex& profiler_mutex() { static std::mutex mu; return mu; }

struct Launch {
    int id; cudaStream_t s; cudaEvent_t a = nullptr, b = nullptr;
    Launch(int id_, cudaStream_t s_) : id(id_), s(s_) {
        std::lock_guard<std::mutex> lock(profiler_mutex());
        Profiler& p = profiler();
        ++p.launches[id];
        if (p.on) { a = p.get(); b = p.get(); if (a) cudaEventRecord(a, s); }
    }
    ~Launch() {
        if (a && b) {
            cudaEventRecord(b, s);
            std::lock_guard<std::mutex> lock(profiler_mutex());
            profiler().recs.push_back({id, a, b});
        }
    }
};

}  // namespace ptq
