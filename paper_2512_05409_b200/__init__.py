"""B200 (sm_100a) SQ-format hot path: encode, hybrid INT4/INT8 GEMM, decode.

The product is the C-ABI shared library built from `csrc/` (declared in
`include/sq.h`); this package is its thin ctypes binding.
"""
from .binding import (  # noqa: F401
    SQ_OK, SQ_ERR_INVALID_ARG, SQ_ERR_UNSUPPORTED, SQ_ERR_NULL_POINTER, SQ_ERR_ALIGNMENT,
    SQ_ERR_ARCH, SQ_ERR_CUDA, SQ_ERR_TIMEOUT, SQ_POS_DYNAMIC, SQ_POS_STATIC, SQ_POS_STATIC_INDEP, SQ_LAYOUT_VERSION,
    SQ_MAX_K, LIBRARY_PATH, SqError, Encoded, Weights, sq_format, sq_encoded, sq_weights,
    make_format, alloc_encoded, alloc_weights, sq_status_string, sq_encoded_sizes,
    sq_weights_sizes, sq_calib_positions, sq_pack_weights, sq_encode, sq_gemm, sq_gemm_ws,
    sq_gemm_workspace_bytes, sq_gemm_static_scratch, SQ_STATIC_SCRATCH_BYTES, sq_decode,
    sq_device_status, sq_device_status_word, raw, FpWeights, sq_fp_pack_weights, sq_fp_encode, sq_fp_gemm, sq_fp_decode, SqWeights, sq_w_encode, sq_w_act_quant, sq_w_gemm,
    sq_encode_a8, sq_gemm_a8, sq_probe_int8_tensor_rate, sq_probe_fp8_tensor_rate, sq_rmsnorm_encode, sq_fp_rmsnorm_encode,
)
from .sharding import row_shard  # noqa: F401,E402
