// Shared plumbing of libadacomp: status handling, launch helpers, small device utilities.
#pragma once

#include <cuda_runtime.h>
#include <atomic>
#include <stdint.h>
#include <stddef.h>

#include "adacomp.h"

namespace adacomp {

extern thread_local int g_last_cuda_error;
extern std::atomic<uint64_t> g_kernel_launches;

inline int cuda_fail(cudaError_t e) {
    g_last_cuda_error = static_cast<int>(e);
    return ADACOMP_ERR_CUDA;
}

#define ADACOMP_CUDA(call)                                         \
    do {                                                           \
        cudaError_t e__ = (call);                                  \
        if (e__ != cudaSuccess) return ::adacomp::cuda_fail(e__);  \
    } while (0)

// Placed after every kernel launch: counts it and turns a launch failure into a status.
#define ADACOMP_LAUNCH_CHECK()                                      \
    do {                                                            \
        ::adacomp::g_kernel_launches.fetch_add(1, std::memory_order_relaxed); \
        ADACOMP_CUDA(cudaGetLastError());                           \
    } while (0)

// Switches to a device for the lifetime of the object and restores the previous one.
struct DeviceGuard {
    int prev = -1;
    bool changed = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int dev) {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != dev) {
            err = cudaSetDevice(dev);
            changed = (err == cudaSuccess);
        }
    }
    ~DeviceGuard() {
        if (changed) cudaSetDevice(prev);
    }
};

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

// Carves aligned sub-buffers out of a caller-provided workspace; with base == nullptr it only
// measures.
struct Carver {
    char* base;
    size_t used = 0;
    explicit Carver(void* b) : base(static_cast<char*>(b)) {}
    template <typename T>
    T* take(size_t count) {
        size_t at = used;
        used = align_up(used + count * sizeof(T));
        return base ? reinterpret_cast<T*>(base + at) : nullptr;
    }
};

// Magnitude key: fp32 bit pattern without the sign bit.  Unsigned order of keys is the order of
// |g| for every non-NaN value (Algorithm 1, SELECT_GRAD: "largest ... in absolute value").
__device__ __forceinline__ uint32_t magnitude_key(float g) { return __float_as_uint(g) & 0x7FFFFFFFu; }

// First device-side error wins; 0 means none.
__device__ __forceinline__ void record_error(int* status_word, int code) { atomicCAS(status_word, 0, code); }

}  // namespace adacomp
