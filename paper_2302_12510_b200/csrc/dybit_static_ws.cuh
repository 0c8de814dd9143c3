// dybit_gemm_static_ws: the GEMM for callers that cannot obtain device memory
// at call time.  Its scratch lives in this library's own image instead of in a
// caller-supplied workspace.
#pragma once

#include "dybit_gemm.cuh"

// Scratch for the expanded operands.  Part of the loaded module: every GPU on
// which a process uses this library sets the bytes aside from module load
// until the process exits, whether or not this entry point is ever called.
static __device__ __align__(256) unsigned char g_static_gemm_ws[DYBIT_STATIC_WS_BYTES + 1024];

namespace dybit {

// The symbol above is only a host-side handle; kernels need the address the
// module was given on the current device.  Looked up once per device.
static dybit_status static_ws_device_pointer(unsigned char **out) {
    static std::atomic<unsigned char *> cached[64];   // filled on first use; a race stores the same address twice
    int dev = 0;
    DYBIT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return DYBIT_ERR_CUDA;
    unsigned char *ptr = cached[dev].load(std::memory_order_acquire);
    if (ptr == nullptr) {
        DYBIT_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_gemm_ws));
        if (ptr == nullptr) return DYBIT_ERR_CUDA;
        cached[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return DYBIT_OK;
}

}  // namespace dybit

extern "C" dybit_status dybit_gemm_static_ws(int64_t M, int64_t N, int64_t K, const void *A, dybit_fmt fa,
                                             const float *scale_a, int64_t lda_bytes, const void *B, dybit_fmt fb,
                                             const float *scale_b, int64_t ldb_bytes, float *C, int64_t ldc,
                                             int32_t *C_raw, void *stream) {
    using namespace dybit;
    const size_t need = dybit_gemm_workspace_bytes(M, N, K, fa, fb);
    if (need == 0) return DYBIT_ERR_INVALID_ARG;
    if (need > (size_t)DYBIT_STATIC_WS_BYTES) return DYBIT_ERR_WORKSPACE;   // problem too large for the built-in scratch
    unsigned char *base = nullptr;
    dybit_status st = static_ws_device_pointer(&base);
    if (st != DYBIT_OK) return st;
    // the GEMM wants 1024-byte alignment; the array carries 1024 spare bytes for that
    unsigned char *ws = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(base) + 1023) & ~uintptr_t(1023));
    return dybit_gemm(M, N, K, A, fa, scale_a, lda_bytes, B, fb, scale_b, ldb_bytes, C, ldc, C_raw, ws,
                      (size_t)DYBIT_STATIC_WS_BYTES, stream);
}
