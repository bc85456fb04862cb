"""B200-native fused W8A8 linear layer: per-token int8 activations x per-channel int8 weights,
int32 accumulation on the tensor cores, dequantization and bias in the GEMM epilogue.

The compute lives in ``libw8a8_linear.so`` (CUDA, sm_100a; C ABI in ``include/w8a8_linear.h``);
``binding`` is the thin ctypes layer over it. The helper modules ``inputs`` (seeded synthetic
tensors), ``roofline`` (work and byte model) and ``dist`` (multi-rank plumbing) hold none of the
method's arithmetic and do not need the CUDA library: importing them, or this package, maps no
native code. The library is loaded the first time a compute entry point (any name exported by
``binding``) is touched, and that raises if it has not been built: there is no CPU fallback.
"""
from __future__ import annotations

import importlib

_BINDING_NAMES = (
    "ACT_BF16", "ACT_INT8", "K_MAX", "STATIC_WORKSPACE_BYTES", "W8A8Error", "alloc_workspace", "config_name",
    "force_config", "int8_check_status", "int8_gemm_i32_debug", "int8_linear_fused", "int8_linear_fused_host",
    "int8_linear_fused_static", "int8_linear_workspace_bytes", "int8_linear_workspace_offsets",
    "int8_quantize_act_per_token", "int8_quantize_weight_per_channel", "num_configs",
    "int8_quantize_act_per_token_smooth", "int8_quantize_weight_per_channel_smooth", "int8_linear_fused_smooth",
    "status_string", "int8_linear_workspace_min_bytes", "int8_linear_plan", "int8_sticky_status",
    "debug_set_wait_limit_ns", "debug_set_starve", "debug_set_small_path", "gemm_clock_stamps", "int8_linear_fused_rowmax",
    "int8_quantize_act_per_token_given_absmax",
)


def __getattr__(name: str):
    # PEP 562: resolved only when somebody asks for a compute entry point
    if name == "binding" or name in _BINDING_NAMES:
        binding = importlib.import_module(".binding", __name__)
        return binding if name == "binding" else getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")


def __dir__():
    return sorted(list(globals()) + list(_BINDING_NAMES) + ["binding"])
