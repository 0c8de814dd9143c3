// placeholder until the tcgen05 GEMM lands
#pragma once
#include "dybit_common.cuh"
extern "C" {
size_t dybit_gemm_workspace_bytes(int64_t, int64_t, int64_t, dybit_fmt, dybit_fmt) { return 0; }
size_t dybit_conv2d_workspace_bytes(const dybit_conv_desc *, dybit_fmt, dybit_fmt) { return 0; }
dybit_status dybit_gemm(int64_t, int64_t, int64_t, const void *, dybit_fmt, const float *, int64_t,
                        const void *, dybit_fmt, const float *, int64_t, float *, int64_t, int32_t *,
                        void *, size_t, void *) { return DYBIT_ERR_UNSUPPORTED; }
dybit_status dybit_conv2d(const dybit_conv_desc *, const void *, dybit_fmt, const float *,
                          const void *, dybit_fmt, const float *, int64_t, float *, int32_t *,
                          void *, size_t, void *) { return DYBIT_ERR_UNSUPPORTED; }
}
