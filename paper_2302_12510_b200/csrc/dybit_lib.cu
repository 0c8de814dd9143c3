// libdybit: single translation unit (the device status word and the kernels
// share one module, so no relocatable device code is needed).
#include "dybit_host.cuh"
#include "dybit_quantize.cuh"
#include "dybit_gemm.cuh"
#include "dybit_gemm_pair.cuh"
#include "dybit_conv_halo.cuh"
#include "dybit_gemm_bdec.cuh"
#include "dybit_static_ws.cuh"
#include "dybit_depthwise.cuh"
