// Internal helpers shared by the translation unit of libdybit (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

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
inline unsigned long long &launch_counter() {
    static unsigned long long n = 0;
    return n;
}

inline dybit_status launch_status() {
    ++launch_counter();
    return cudaGetLastError() == cudaSuccess ? DYBIT_OK : DYBIT_ERR_CUDA;
}

struct ProfileEvents {
    cudaEvent_t start = nullptr, stop = nullptr;
};
inline ProfileEvents &profile_events() {
    static thread_local ProfileEvents ev;
    return ev;
}

// Device status word: 0 = fine; otherwise (site << 8) | 1 of the first bounded
// wait that expired.  Kernels only ever OR a value in.
__device__ unsigned int g_device_status = 0;

// Number of SMs of the current device (cached per device id).
int sm_count();

}  // namespace dybit
