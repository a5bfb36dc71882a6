// Rounding masks of the paper's baselines for the higher-bit weights: BitShift (always round down), rounding
// up, and round-to-nearest (RTN, ties to the even neighbour).  NestQuant itself takes the mask from an adaptive
// rounding optimiser (SQuant), which is outside this library; these three are the rows it is compared with in the
// ablation of the rounding and in the numerical-error table, and they make nq_decompose usable on its own.
// Element-wise and bandwidth-bound: one thread per 16 weights when the pointers and pitches allow 128-bit accesses.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/nq.h"
#include "nq_internal.cuh"

namespace {

__device__ __forceinline__ uint32_t mask_of(int w, int l, int mode) {
    if (mode == NQ_ROUND_DOWN) return 0u;
    if (mode == NQ_ROUND_UP) return 1u;
    const int down = w >> l;                       // arithmetic shift = floor
    const int rem = w - (down << l);               // 0 .. 2^l - 1
    const int two_rem = 2 * rem, two_l = 1 << l;
    if (two_rem > two_l) return 1u;
    if (two_rem < two_l) return 0u;
    return (uint32_t)(down & 1);                   // tie: go to the even neighbour
}

__global__ void __launch_bounds__(256) rounding_mask_kernel(const int8_t* __restrict__ w, int64_t ld_w, int64_t rows,
                                                            int64_t cols, int l, int mode, uint8_t* __restrict__ mask,
                                                            int64_t ld_m, int vec) {
    const int64_t chunks_per_row = (cols + 15) >> 4;
    const int64_t total = rows * chunks_per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / chunks_per_row, c0 = (i - row * chunks_per_row) << 4;
        const int8_t* src = w + row * ld_w + c0;
        uint8_t* dst = mask + row * ld_m + c0;
        if (vec && c0 + 16 <= cols) {
            const uint4 v = *reinterpret_cast<const uint4*>(src);
            const uint32_t in[4] = {v.x, v.y, v.z, v.w};
            uint32_t out[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t o = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) o |= mask_of((int)(int8_t)(in[q] >> (8 * b)), l, mode) << (8 * b);
                out[q] = o;
            }
            *reinterpret_cast<uint4*>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
        } else {
            for (int j = 0; j < 16 && c0 + j < cols; ++j) dst[j] = (uint8_t)mask_of((int)src[j], l, mode);
        }
    }
}

}  // namespace

extern "C" int nq_rounding_mask(const int8_t* w_int, int64_t ld_w, int64_t rows, int64_t cols, int n_bits, int h_bits,
                                int mode, uint8_t* mask_out, int64_t ld_mask, void* stream) {
    if (rows < 0 || cols < 0) return NQ_ERR_INVALID_ARG;
    if (n_bits < 2 || n_bits > 8 || h_bits < 1 || h_bits >= n_bits) return NQ_ERR_UNSUPPORTED;
    if (mode != NQ_ROUND_DOWN && mode != NQ_ROUND_UP && mode != NQ_ROUND_NEAREST) return NQ_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return NQ_OK;
    if (!w_int || !mask_out || ld_w < cols || ld_mask < cols) return NQ_ERR_INVALID_ARG;
    const int vec = ((reinterpret_cast<uintptr_t>(w_int) | reinterpret_cast<uintptr_t>(mask_out)) & 15) == 0 &&
                    (ld_w & 15) == 0 && (ld_mask & 15) == 0;
    const int64_t chunks = rows * ((cols + 15) >> 4);
    const int64_t need = (chunks + 255) / 256, cap = (int64_t)nq::sm_count() * 32;
    rounding_mask_kernel<<<(unsigned)(need < cap ? need : cap), 256, 0, (cudaStream_t)stream>>>(
        w_int, ld_w, rows, cols, n_bits - h_bits, mode, mask_out, ld_mask, vec);
    return cudaGetLastError() == cudaSuccess ? NQ_OK : NQ_ERR_CUDA;
}
