// Implicit-GEMM convolution entry points (under construction: the contraction core is shared with the GEMM).
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/nq.h"

extern "C" {

int64_t nq_conv_workspace_bytes(const nq_conv_desc* desc) {
    if (!desc) return -1;
    return 0;
}

int nq_conv_implicit_gemm(const int8_t*, const void*, int64_t, int, int, int, const nq_conv_desc*, const float*, float,
                          const float*, int32_t*, void*, int, void*, int64_t, void*) {
    return NQ_ERR_UNSUPPORTED;
}

}  // extern "C"
