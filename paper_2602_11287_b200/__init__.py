"""HiF4 (HiFloat4) W4A4 linear-layer hot path for B200: Python names of the C ABI in include/hif4.h."""
from .binding import (  # noqa: F401
    EXPORTED_SYMBOLS, HIF4_BF16, HIF4_FMT_HIF4, HIF4_FMT_MXFP4, HIF4_FMT_NVFP4, HIF4_FMT_NVFP4_PTS, hif4_mse_roundtrip, hif4_mse_workspace, HIF4_FP16, HIF4_FP32, HIF4_RHA, HIF4_RNE, LIB_PATH, UNIT_BYTES, UNIT_ELEMS, Hif4Error,
    hif4_dequantize, hif4_gemm, hif4_gemm_workspace, hif4_grouped_gemm, hif4_grouped_gemm_noalloc, hif4_grouped_gemm_noalloc_capacity, hif4_grouped_gemm_workspace,
    hif4_last_device_status, hif4_linear, hif4_linear_workspace, hif4_packed_bytes, hif4_quantize, hif4_quantize_transposed, hif4_debug_set_gemm_path, hif4_debug_wait_timeout, launch_count, lib, status_string,
)
