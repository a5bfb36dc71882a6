"""B200-native (sm_100a) implementation of NestQuant's nested-integer hot path.

The work happens in ``libnq_b200.so`` (hand-written CUDA behind the C boundary of ``include/nq.h``);
``binding`` marshals torch tensors into it.  Nothing is loaded at import time: the first call
loads the library and raises ``NqLibraryError`` if it has not been built -- there is no fallback.
"""
from .binding import (  # noqa: F401
    BatchPlan, NqError, NqLibraryError, EXPORTS, NQ_BF16, NQ_F32, lib, nq_batch_plan, nq_conv_desc,
    nq_conv_implicit_gemm, nq_conv_implicit_gemm_static, nq_conv_workspace_bytes, NQ_CONV_STATIC_SCRATCH_BYTES, nq_decompose, nq_device_status, nq_drop_low,
    nq_drop_low_batched, nq_gemm_full, nq_gemm_part, nq_low_bits, nq_pack, nq_packed_bytes,
    nq_packed_row_bytes, nq_recompose, nq_recompose_batched, nq_tensor_desc, nq_unpack, status_str,
    nq_word64_row_words, nq_word64_to_sliced, nq_sliced_to_word64,
    nq_gemm_full_q8, nq_gemm_part_q8, nq_conv_implicit_gemm_q8, nq_gemm_nested, nq_conv_implicit_gemm_nested, nq_gemm_nested_q8,
    nq_conv_implicit_gemm_nested_q8,
    nq_i8_mma_ceiling, nq_debug_set, NQ_DEBUG_PLAIN_STORES, NQ_DEBUG_PACKED_RING,
    nq_conv_implicit_gemm_q8_res, nq_conv_implicit_gemm_nested_q8_res, nq_maxpool_nhwc_i8, nq_avgpool_requant_nhwc_i8,
    nq_rounding_mask, NQ_ROUND_DOWN, NQ_ROUND_UP, NQ_ROUND_NEAREST,
)
