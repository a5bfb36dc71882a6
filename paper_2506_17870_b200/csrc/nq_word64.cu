// Converters between the paper's packed-bit tensor and the library's sliced layout.
//
// The paper ("Deployment": packed-bit tensors) stores a k-bit weight tensor as unsigned 64-bit words with
// 64 // k fields each, field j at bits [j*k, j*k + k), the unused top bits zero (twenty-one 3-bit or twelve
// 5-bit weights per word).  That is the format a model arrives in; the kernels of this library work on the
// sliced layout of nq.h.  Both directions are plain element-wise moves of k-bit two's-complement fields:
//   word64 -> sliced   one thread per 32-element unit, in nq_codec.cu beside the slice cutter it shares with
//                      the codec kernels
//   sliced -> word64   one thread per output word: gathers its 64 // k fields out of the slices
// They are conversion utilities (run once per model), written for clarity; the hot codec is nq_codec.cu.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/nq.h"
#include "nq_internal.cuh"

namespace {

// Where slice `s` (a power of two) keeps the bits of element e of a row's 128: byte offset inside the row's 16 * s
// bytes of that slice and shift inside that byte (the first of the 8/s fields that share a byte sits in its top bits).
__device__ __forceinline__ void slice_place(int s, int e, int& byte_off, int& shift) {
    const int unit = e >> 5, q = (e & 31) >> 2, lane = e & 3;
    const int per_byte = 8 / s;
    const int word = q / per_byte, sub = q - word * per_byte;
    byte_off = ((unit * s + word) << 2) + lane;
    shift = 8 - s * sub - s;
}

template <int BITS>
__global__ void __launch_bounds__(256) sliced_to_word64_kernel(const uint8_t* __restrict__ packed, int64_t rows,
                                                               int64_t cols, uint64_t* __restrict__ words) {
    constexpr int PER = 64 / BITS;
    const int64_t groups_per_row = (cols + 127) >> 7;
    const int64_t row_words = (cols + PER - 1) / PER;
    const int64_t total = rows * row_words;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = i / row_words, wd = i - row * row_words;
        uint64_t out = 0;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int64_t c = wd * PER + j;
            if (c >= cols) break;
            // block (row / 128, column group), 2048 * BITS bytes; in it the slices, each 128 rows of 16 * s bytes
            const uint8_t* block = packed + ((row >> 7) * groups_per_row + (c >> 7)) * 2048 * BITS;
            const int e = (int)(c & 127), r = (int)(row & 127);
            uint32_t field = 0;
            int slice_base = 0;
#pragma unroll
            for (int s = 8; s >= 1; s >>= 1) {
                if (!(BITS & s)) continue;
                int off, sh;
                slice_place(s, e, off, sh);
                field = (field << s) | ((uint32_t)(block[slice_base + r * 16 * s + off] >> sh) & ((1u << s) - 1u));
                slice_base += 2048 * s;
            }
            out |= (uint64_t)field << (j * BITS);
        }
        words[i] = out;
    }
}

inline int blocks_for(int64_t threads) {
    const int64_t need = (threads + 255) / 256;
    const int64_t cap = (int64_t)nq::sm_count() * 16;
    return (int)(need < cap ? need : cap);
}

template <int BITS>
int launch_from_sliced(const void* src, int64_t rows, int64_t cols, void* dst, cudaStream_t s) {
    const int64_t n = rows * ((cols + 64 / BITS - 1) / (64 / BITS));
    sliced_to_word64_kernel<BITS><<<blocks_for(n), 256, 0, s>>>(static_cast<const uint8_t*>(src), rows, cols,
                                                                static_cast<uint64_t*>(dst));
    return cudaGetLastError() == cudaSuccess ? NQ_OK : NQ_ERR_CUDA;
}

int convert(bool to_sliced, const void* src, int bits, int64_t rows, int64_t cols, void* dst, void* stream) {
    if (rows < 0 || cols < 0) return NQ_ERR_INVALID_ARG;
    if (bits < 1 || bits > 8) return NQ_ERR_UNSUPPORTED;
    if (rows == 0 || cols == 0) return NQ_OK;
    if (!src || !dst) return NQ_ERR_INVALID_ARG;
    const void* sliced = to_sliced ? dst : src;
    const void* w64 = to_sliced ? src : dst;
    if ((reinterpret_cast<uintptr_t>(sliced) & 15) || (reinterpret_cast<uintptr_t>(w64) & 7)) return NQ_ERR_ALIGNMENT;
    cudaStream_t s = (cudaStream_t)stream;
    if (to_sliced)
        return nq::word64_to_sliced_launch(static_cast<const uint64_t*>(src), bits, rows, cols, static_cast<uint8_t*>(dst), s);
    switch (bits) {
        case 1: return launch_from_sliced<1>(src, rows, cols, dst, s);
        case 2: return launch_from_sliced<2>(src, rows, cols, dst, s);
        case 3: return launch_from_sliced<3>(src, rows, cols, dst, s);
        case 4: return launch_from_sliced<4>(src, rows, cols, dst, s);
        case 5: return launch_from_sliced<5>(src, rows, cols, dst, s);
        case 6: return launch_from_sliced<6>(src, rows, cols, dst, s);
        case 7: return launch_from_sliced<7>(src, rows, cols, dst, s);
        default: return launch_from_sliced<8>(src, rows, cols, dst, s);
    }
}

}  // namespace

extern "C" {

int64_t nq_word64_row_words(int64_t cols, int bits) {
    if (cols < 0 || bits < 1 || bits > 8) return -1;
    const int64_t per = 64 / bits;
    return (cols + per - 1) / per;
}

int nq_word64_to_sliced(const uint64_t* words, int bits, int64_t rows, int64_t cols, void* packed_out, void* stream) {
    return convert(true, words, bits, rows, cols, packed_out, stream);
}

int nq_sliced_to_word64(const void* packed, int bits, int64_t rows, int64_t cols, uint64_t* words_out, void* stream) {
    return convert(false, packed, bits, rows, cols, words_out, stream);
}

}  // extern "C"
