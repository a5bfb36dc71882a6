// Host-side helpers shared by the translation units of the library (not part of the C boundary).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace nq {

// SM count of the current device (cached per device index).
int sm_count();

// Device-side record of a bounded wait that gave up: word 0 = non-zero code of the wait, word 1 = detail.
// Defined in nq_runtime.cu; kernels get its address through status_word().
unsigned int* status_word();

// The paper's 64-bit packed words -> sliced layout (kernel beside the codec, whose slice cutter it uses).
int word64_to_sliced_launch(const uint64_t* words, int bits, int64_t rows, int64_t cols, uint8_t* packed, cudaStream_t s);

}  // namespace nq

