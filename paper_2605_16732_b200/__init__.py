"""DiRotQ rotation-aware W4A4 linear layer for B200: CUDA library + thin binding."""
from .binding import (  # noqa: F401
    DirotqError, Layer, alloc_workspace, dirotq_int_gemm_debug, dirotq_layer_bytes, dirotq_layer_export,
    dirotq_linear, dirotq_linear_host, dirotq_linear_noalloc, dirotq_prepare_layer, dirotq_prepare_scratch_bytes, dirotq_rotate_quantize, dirotq_w4a4_gemm,
    dirotq_workspace_bytes, dirotq_workspace_export, dirotq_workspace_status, lib,
)
