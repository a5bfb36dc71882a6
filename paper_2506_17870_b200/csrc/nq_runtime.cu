// Small runtime pieces: status text, SM count, and the device-side record of expired waits.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/nq.h"
#include "nq_internal.cuh"

namespace nq {

__device__ unsigned int g_status_word[4];

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

unsigned int* status_word() {
    static unsigned int* cached[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cached[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
        cached[dev] = static_cast<unsigned int*>(p);
    }
    return cached[dev];
}

}  // namespace nq

extern "C" {

const char* nq_status_str(int status) {
    switch (status) {
        case NQ_OK: return "ok";
        case NQ_ERR_INVALID_ARG: return "invalid argument";
        case NQ_ERR_UNSUPPORTED: return "unsupported nesting or shape";
        case NQ_ERR_ALIGNMENT: return "pointer or pitch alignment";
        case NQ_ERR_WORKSPACE: return "workspace missing or too small";
        case NQ_ERR_CUDA: return "CUDA call failed";
        case NQ_ERR_TIMEOUT: return "bounded device wait expired";
        default: return "unknown status";
    }
}

int nq_device_status(void* stream, int* where_out) {
    unsigned int* word = nq::status_word();
    if (!word) return NQ_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return NQ_ERR_CUDA;
    unsigned int host[4] = {0, 0, 0, 0};
    if (cudaMemcpy(host, word, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess) return NQ_ERR_CUDA;
    if (where_out) *where_out = (int)host[0];
    if (host[0] == 0) return NQ_OK;
    if (cudaMemset(word, 0, sizeof(host)) != cudaSuccess) return NQ_ERR_CUDA;
    return NQ_ERR_TIMEOUT;
}

}  // extern "C"
