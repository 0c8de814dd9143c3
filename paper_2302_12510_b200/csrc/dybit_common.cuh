// Internal helpers shared by the translation unit of libdybit (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "dybit.h"

namespace dybit {

// Magnitude bits of a format: a signed code spends its top bit on the sign.
__host__ __device__ inline int mag_bits(dybit_fmt f) { return f.is_signed ? f.bits - 1 : f.bits; }

inline bool fmt_ok(dybit_fmt f) {
    return f.bits >= 2 && f.bits <= 8 && (f.is_signed == 0 || f.is_signed == 1);
}

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

#define DYBIT_CUDA_TRY(expr)                         \
    do {                                             \
        cudaError_t e__ = (expr);                    \
        if (e__ != cudaSuccess) {                    \
            (void)cudaGetLastError();                \
            return DYBIT_ERR_CUDA;                   \
        }                                            \
    } while (0)

// Every kernel launch of the library is followed by launch_status(), which
// also counts it.
inline std::atomic<unsigned long long> &launch_counter() {
    static std::atomic<unsigned long long> n{0};
    return n;
}

inline dybit_status launch_status() {
    launch_counter().fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? DYBIT_OK : DYBIT_ERR_CUDA;
}

// Every kernel of the library is launched with programmatic stream serialization: a kernel may be
// scheduled while its predecessor in the stream is still draining, runs its prologue, and then blocks in
// pdl_enter() until the predecessor has completed and its writes are visible.  pdl_enter() also releases
// the kernel's own successor, so at most one successor is ever waiting.  Chains of short dependent kernels
// (absmax -> quantize -> expand -> GEMM) overlap their launch and ramp-up this way.
template <typename... KArgs, typename... Args>
inline void launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    (void)cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

__device__ __forceinline__ void pdl_enter() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

struct ProfileEvents {
    cudaEvent_t start = nullptr, stop = nullptr;
    unsigned long long *clock = nullptr;      // device pair {first start, last end} in %globaltimer ns
};
inline ProfileEvents &profile_events() {
    static thread_local ProfileEvents ev;
    return ev;
}

// Device status word: 0 = fine; otherwise (site << 8) | 1 of the first bounded
// wait that expired.  Kernels only ever OR a value in.
__device__ unsigned int g_device_status = 0;

// Range checks of the debug build (-DDYBIT_DEBUG_BOUNDS, libdybit_debug.so): global-memory stores whose extent the
// kernel knows are wrapped in `if (DYBIT_CHECK(index condition, site))`.  A failing check skips the access and ORs
// (site << 8) | 2 into the status word (dybit_last_device_status then reports DYBIT_ERR_DEVICE_BOUNDS); nothing
// traps.  In the normal build the macro is the constant true and the condition is not evaluated.
#ifdef DYBIT_DEBUG_BOUNDS
__device__ __forceinline__ bool debug_range_ok(bool cond, unsigned site) {
    if (!cond) atomicOr(&g_device_status, (site << 8) | 2u);
    return cond;
}
#define DYBIT_CHECK(cond, site) ::dybit::debug_range_ok((cond), (site))
#else
#define DYBIT_CHECK(cond, site) true
#endif

// Number of SMs of the current device (cached per device id).
int sm_count();

}  // namespace dybit
