// Shared host/device helpers of the quantizer library (status word, launch checks, workspace carving).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

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

}  // namespace ptq
