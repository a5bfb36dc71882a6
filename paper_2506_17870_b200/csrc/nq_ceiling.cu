// Issue-only ceiling of the tensor path the contraction kernels use: tcgen05.mma kind::i8 on CTA pairs
// (cta_group::2, 256 x 256 x 32 per instruction), operands parked in shared memory, accumulators in tensor
// memory, no loads from global memory, no epilogue.  What a launch of this kernel sustains is the most any
// INT8 contraction built on these instructions can reach on the same GPU under the same power limit; the
// benchmark divides the GEMM rates by it.
//
// One CTA pair per two SMs.  Each CTA fills a ring of operand stages (the full-bit kernel's footprint: six
// stages of 128 rows x 128 bytes for A and for its half of B) with small signed pseudo-random bytes -- the
// toggle rate of the operands sets the power draw, and with it the clock -- and the leader's issuing thread
// then runs `stage_iters` stages of four MMAs each, walking the ring and alternating between the two
// accumulators every 64 stages, exactly the instruction stream of the contraction kernel's issuing thread
// without its waits.  One commit at the end tells both CTAs that everything has completed; that wait is bounded.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/nq.h"
#include "nq_contraction_pair.cuh"
#include "nq_internal.cuh"

namespace nq {
namespace {

constexpr int kCeilStages = kPairStagesFull;
constexpr int kCeilThreads = 128;
constexpr int kCeilSmem = kCeilStages * (a_stage_bytes() + b_stage_bytes(kPairBN / 2)) + 64 + 1024;

__global__ void __launch_bounds__(kCeilThreads, 1) i8_mma_ceiling_kernel(long long stage_iters, unsigned int* status) {
    using namespace sm100;
    constexpr int A_BYTES = a_stage_bytes();
    constexpr int B_BYTES = b_stage_bytes(kPairBN / 2);
    constexpr uint32_t TMEM_COLS = 2 * kPairBN;
    constexpr uint32_t IDESC = idesc_i8(2 * kBM, kPairBN);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sB = sA + kCeilStages * A_BYTES;
    uint64_t* done = reinterpret_cast<uint64_t*>(sB + kCeilStages * B_BYTES);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(done + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();

    // operands: bytes in [-63, 63], the difference of two 6-bit hash fields (a bell shape like quantised weights)
    uint32_t* words = reinterpret_cast<uint32_t*>(smem);
    const int n_words = kCeilStages * (A_BYTES + B_BYTES) / 4;
    for (int i = threadIdx.x; i < n_words; i += kCeilThreads) {
        uint32_t w = 0;
        for (int b = 0; b < 4; ++b) {
            uint32_t x = (uint32_t)(i * 4 + b) * 2654435761u + blockIdx.x * 40503u;
            x ^= x >> 15; x *= 2246822519u; x ^= x >> 13;
            const int v = (int)(x & 63u) - (int)((x >> 6) & 63u);
            w |= (uint32_t)(v & 0xff) << (8 * b);
        }
        words[i] = w;
    }
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(done), 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    fence_proxy_async_smem();                 // generic-proxy writes -> visible to tcgen05.mma
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 1 && lane == 0) {
        if (rank == 0) {
            uint32_t s = 0;
            for (uint32_t it = 0; it < (uint32_t)stage_iters; ++it, s = (s + 1 == kCeilStages) ? 0u : s + 1) {
                const uint32_t d_tmem = tmem_base + ((it >> 6) & 1u) * kPairBN;
                const uint64_t da = smem_desc_sw128(smem_u32(sA + s * A_BYTES));
                const uint64_t db = smem_desc_sw128(smem_u32(sB + s * B_BYTES));
#pragma unroll
                for (int k = 0; k < kBK / 32; ++k) mma_i8_pair(d_tmem, da + 2 * k, db + 2 * k, IDESC, (it & 63) != 0 || k != 0);
            }
            mma_commit_pair(smem_u32(done));  // arrives in both CTAs once every MMA above has completed
        }
        (void)mbar_wait_cluster(smem_u32(done), 0, abort_flag, status, 0x300u);
    }

    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

}  // namespace
}  // namespace nq

extern "C" int nq_i8_mma_ceiling(int64_t stage_iters, double* ops_out, void* stream) {
    using namespace nq;
    // a launch must end well inside the bounded wait of about a second: 2^21 stages are about half a second
    if (stage_iters < 1 || stage_iters > (1ll << 21)) return NQ_ERR_INVALID_ARG;
    unsigned int* status = status_word();
    if (!status) return NQ_ERR_CUDA;
    static int configured[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return NQ_ERR_CUDA;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(i8_mma_ceiling_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kCeilSmem) != cudaSuccess)
            return NQ_ERR_CUDA;
        configured[dev] = 1;
    }
    const int pairs = sm_count() / 2;
    if (pairs < 1) return NQ_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs, 1, 1);
    cfg.blockDim = dim3(kCeilThreads, 1, 1);
    cfg.dynamicSmemBytes = kCeilSmem;
    cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, i8_mma_ceiling_kernel, (long long)stage_iters, status) != cudaSuccess) {
        (void)cudaGetLastError();
        return NQ_ERR_CUDA;
    }
    // per stage and pair: four instructions of 256 x 256 x 32 multiply-accumulates, two operations each
    if (ops_out) *ops_out = (double)pairs * (double)stage_iters * 4.0 * 2.0 * 256.0 * 256.0 * 32.0;
    return NQ_OK;
}
