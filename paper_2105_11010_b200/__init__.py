"""B200 (sm_100a) SPARQ hot path: thin Python binding over the C-ABI library.

Every step of the path runs in the library's CUDA kernels; this package only
marshals arguments (torch tensors are used for device memory and streams).
There is no CPU fallback: importing the binding without the built shared
library raises.
"""
from ._binding import (  # noqa: F401
    SparqParams,
    SparqError,
    MODE_NONE, MODE_BSPARQ, MODE_VSPARQ,
    ROUND_TRUNCATE, ROUND_NEAREST,
    SET_5OPT, SET_3OPT, SET_2OPT, SET_6OPT, SET_7OPT,
    library_path, load_library,
    sparq_quantize, sparq_gemm_s8, sparq_conv2d_nhwc_s8,
    sparq_quantize_host, sparq_gemm_s8_host, sparq_conv2d_nhwc_s8_host,
    sparq_gemm_s8_static, STATIC_SCRATCH_BYTES,
    sparq_packed_ctrl_bits, sparq_pack, sparq_unpack,
    sparq_sparse24_expanded_k, sparq_sparse24_expand_weights, sparq_sparse24_expand_activations,
    sparq_gemm_s8_sparse24,
    sparq_absmax, sparq_quantize_act_u8, sparq_quantize_weight_s8, DTYPE_F32, DTYPE_BF16,
    sparq_check, sparq_last_error, sparq_shutdown, sparq_selftest_wait_timeout, sparq_selftest_mma_rate,
)
