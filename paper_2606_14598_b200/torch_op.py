"""The fused W8A8 linear as a PyTorch custom operator and a drop-in module.

The paper lists a graph-safe custom operator as its first piece of future work (its own integration disabled
the graph tracer around every quantized linear, and the ablation with the compiler then broke the graph at each
of them). Registered through ``torch.library`` with a shape-only ("fake") implementation, the operator below is
opaque to the tracer but not a graph break: ``torch.compile(fullgraph=True)`` traces through modules that call it,
and because the library call allocates nothing and only enqueues on the current stream, the compiled function can
also be replayed from a CUDA graph.

Marshalling only: the operator's body is one call of the C ABI (``int8_linear_fused`` on bf16 activations); the
workspace it hands over is a torch allocation made inside the operator.
"""
from __future__ import annotations

import torch

from . import binding

__all__ = ["linear_fused", "W8A8Linear"]


@torch.library.custom_op("w8a8_b200::linear_fused", mutates_args=())
def linear_fused(A: torch.Tensor, qw: torch.Tensor, s_ch: torch.Tensor, bias: torch.Tensor | None) -> torch.Tensor:
    """bf16 [..., K] activations x int8 [N, K] per-channel weights -> bf16 [..., N] (quantize, int8 GEMM, dequantize)."""
    lead = A.shape[:-1]
    A2 = A.reshape(-1, A.shape[-1])
    if A2.stride(-1) != 1:
        A2 = A2.contiguous()
    M, K = A2.shape
    N = qw.shape[0]
    out = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
    if M > 0:
        ws = binding.alloc_workspace(M, N, K, binding.ACT_BF16, A.device)
        binding.int8_linear_fused(A2, qw, s_ch, bias, out=out, workspace=ws)
    return out.reshape(*lead, N)


@linear_fused.register_fake
def _linear_fused_fake(A, qw, s_ch, bias):
    torch._check(A.dtype == torch.bfloat16, lambda: "activations must be bf16")
    torch._check(qw.dtype == torch.int8 and qw.dim() == 2, lambda: "weights must be int8 [N, K]")
    torch._check(A.shape[-1] == qw.shape[1], lambda: "K mismatch")
    return A.new_empty((*A.shape[:-1], qw.shape[0]), dtype=torch.bfloat16)


class W8A8Linear(torch.nn.Module):
    """Drop-in replacement of an ``nn.Linear`` forward: weights are quantized once per output channel (on the
    device, by the library), activations per token on every call."""

    def __init__(self, qw: torch.Tensor, s_ch: torch.Tensor, bias: torch.Tensor | None = None):
        super().__init__()
        self.register_buffer("qw", qw)
        self.register_buffer("s_ch", s_ch)
        self.register_buffer("bias", bias)

    @classmethod
    def from_float(cls, weight: torch.Tensor, bias: torch.Tensor | None = None) -> "W8A8Linear":
        """weight: fp32 [N, K] on the CUDA device; bias: fp32 [N] or None."""
        qw, s_ch = binding.int8_quantize_weight_per_channel(weight.float().contiguous())
        return cls(qw, s_ch, None if bias is None else bias.float().contiguous())

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        return linear_fused(x, self.qw, self.s_ch, self.bias)
