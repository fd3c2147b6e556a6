"""B200-native MXFP4 quantized linear layer (TetraJet, arxiv 2502.20853): Python face of libmxfp4.so."""
from .binding import (  # noqa: F401
    DEV_NONFINITE, DEV_SMEM_LAYOUT, DEV_TIMEOUT, EXPORTS, HOOK_GELU, HOOK_IDENTITY, HOOK_MULTIPLY, Epilogue, gemm_quant, LIB_PATH, OUT_BF16, OUT_FP32, ROUND_NEAREST, ROUND_STOCHASTIC,
    SCALE_FLOOR, SCALE_TRUNCATION_FREE, STATIC_SCRATCH_BYTES, LinearCtx, MxError, OscState, QMat, dequantize, gemm, gemm_static,
    gemm_chain_mmas, gemm_wait_selftest, launch_count, gemm_workspace_bytes, quantize_wait_selftest, lib, linear_bwd, linear_fwd, linear_workspace_bytes, new_status, qema_quantize, qramp_adamw, qramp_detect, quant_conf_hist, change_sums, mma_issue_ceiling,
    quantize, quantize_2axis, quantize_chain, quantize_t, scale_bytes, scale_offset,
)
