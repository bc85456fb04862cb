"""B200-native fused W8A8 linear layer: per-token int8 activations x per-channel int8 weights,
int32 accumulation on the tensor cores, dequantization and bias in the GEMM epilogue.

The compute lives in ``libw8a8_linear.so`` (CUDA, sm_100a; C ABI in ``include/w8a8_linear.h``);
this package is the thin binding plus the synthetic-input and work-model helpers.
"""
from .binding import (  # noqa: F401
    ACT_BF16, ACT_INT8, K_MAX, W8A8Error, alloc_workspace, config_name, force_config, int8_check_status,
    int8_gemm_i32_debug, int8_linear_fused, int8_linear_fused_host, int8_linear_fused_static, int8_linear_workspace_bytes,
    int8_linear_workspace_offsets, int8_quantize_act_per_token, int8_quantize_weight_per_channel, num_configs,
    int8_quantize_act_per_token_smooth, int8_quantize_weight_per_channel_smooth, int8_linear_fused_smooth,
    status_string, int8_linear_workspace_min_bytes, int8_linear_plan,
)
