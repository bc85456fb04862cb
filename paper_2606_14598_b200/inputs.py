"""Seeded synthetic inputs shaped like a diffusion transformer's linear layers.

This module only draws numbers. It holds none of the W8A8 method's arithmetic
(no quantizer, no matmul, no dequantization): the CUDA library and the CPU
oracle each receive the tensors made here and do their own work on them.

Recipe (stand-ins for the paper's activations and weights, which are not
available): activations are N(0,1) cast to bf16, with 1% of the K input
channels multiplied by 20 before the cast (outlier channels, picked by a seeded
permutation); the MLP down-projection's activations are GELU(z), z ~ N(0,1),
cast to bf16; weights are fp32 N(0, 0.02^2); bias is fp32 N(0, 0.01^2).
Every tensor comes from its own counter-based Philox stream keyed by
(seed, linear name, tensor id), so a tensor's bits depend on nothing but its own
key and shape.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class LinearSpec:
    """One linear layer of the workload: out[M,N] = A[M,K] @ W[N,K]^T + bias[N]."""
    name: str
    M: int
    K: int
    N: int
    act: str = "normal"          # "normal" | "gelu"
    outlier_frac: float = 0.01   # share of the K channels scaled up
    outlier_mult: float = 20.0
    bias: bool = True

    @property
    def ops(self) -> int:
        return 2 * self.M * self.N * self.K


# The five benchmark configurations (M, K, N as in out[M,N] = A[M,K] W[N,K]^T).
CONFIGS: dict[str, list[LinearSpec]] = {
    # single small linear, no outliers
    "c1": [LinearSpec("c1", 128, 256, 256, outlier_frac=0.0)],
    # attention out-projection at 768px: 2304 image + 512 text tokens
    "c2": [LinearSpec("c2_attn_out", 2816, 3072, 3072)],
    # fused QKV projection at 1024px: 4096 image + 512 text tokens
    "c3": [LinearSpec("c3_qkv", 4608, 3072, 9216)],
    # MLP up and down at 1024px
    "c4": [LinearSpec("c4_mlp_up", 4608, 3072, 12288),
           LinearSpec("c4_mlp_down", 4608, 12288, 3072, act="gelu", outlier_frac=0.0)],
    # all linears of one block at 1024px with the two guidance branches stacked (M = 9216)
    "c5": [LinearSpec("c5_qkv", 9216, 3072, 9216),
           LinearSpec("c5_attn_out", 9216, 3072, 3072),
           LinearSpec("c5_mlp_up", 9216, 3072, 12288),
           LinearSpec("c5_mlp_down", 9216, 12288, 3072, act="gelu", outlier_frac=0.0),
           LinearSpec("c5_adaln", 2, 3072, 18432, outlier_frac=0.0)],
    # The paper's own model (Method, "Target architecture": hidden 4608, MLP 12288, five distinct GEMM shapes
    # (N, K)) at the in-model token count of 1024px (Results: M ~ 4110), rounded up to a multiple of 2.
    "paper": [LinearSpec("paper_qkv", 4110, 4608, 13824),
              LinearSpec("paper_attn_out", 4110, 4608, 4608),
              LinearSpec("paper_ffn_up", 4110, 4608, 12288),
              LinearSpec("paper_ffn_down", 4110, 12288, 4608, act="gelu", outlier_frac=0.0),
              LinearSpec("paper_llm_proj", 4110, 53248, 4608)],
}


def _rng(seed: int, name: str, tensor_id: int) -> np.random.Generator:
    key = (int(seed) & 0xFFFFFFFF) << 32 | zlib.crc32(name.encode())
    return np.random.Generator(np.random.Philox(key=[key, tensor_id]))


def _normal_f32(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(size=shape, dtype=np.float32)


def _gelu_erf(z: np.ndarray) -> np.ndarray:
    # exact (erf) GELU of the draw; an input transform, evaluated in float64
    from scipy.special import erf
    z64 = z.astype(np.float64)
    return (0.5 * z64 * (1.0 + erf(z64 / np.sqrt(2.0)))).astype(np.float32)


def outlier_channels(spec: LinearSpec, seed: int = 0) -> np.ndarray:
    """Indices of the K channels that carry the outlier multiplier (sorted)."""
    n = int(round(spec.outlier_frac * spec.K))
    if n <= 0:
        return np.zeros((0,), np.int64)
    perm = _rng(seed, spec.name, 3).permutation(spec.K)
    return np.sort(perm[:n]).astype(np.int64)


def make_activations(spec: LinearSpec, seed: int = 0, rows: slice | None = None) -> torch.Tensor:
    """bf16 [M,K] activations (CPU tensor). ``rows`` keeps only a row slice of them."""
    x = _normal_f32(_rng(seed, spec.name, 0), (spec.M, spec.K))
    if rows is not None:
        x = x[rows]
    if spec.act == "gelu":
        x = _gelu_erf(x)
    elif spec.act != "normal":
        raise ValueError(spec.act)
    ch = outlier_channels(spec, seed)
    if ch.size:
        x[:, ch] *= np.float32(spec.outlier_mult)
    return torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16)


def make_weight(spec: LinearSpec, seed: int = 0) -> torch.Tensor:
    """fp32 [N,K] weights, N(0, 0.02^2)."""
    w = _normal_f32(_rng(seed, spec.name, 1), (spec.N, spec.K))
    w *= np.float32(0.02)
    return torch.from_numpy(w)


def make_bias(spec: LinearSpec, seed: int = 0) -> torch.Tensor | None:
    """fp32 [N] bias, N(0, 0.01^2); None when the layer has no bias."""
    if not spec.bias:
        return None
    b = _normal_f32(_rng(seed, spec.name, 2), (spec.N,))
    b *= np.float32(0.01)
    return torch.from_numpy(b)


def make_linear(spec: LinearSpec, seed: int = 0) -> dict:
    """All host tensors of one linear: {'A': bf16 [M,K], 'W': fp32 [N,K], 'bias': fp32 [N] | None}."""
    return {"A": make_activations(spec, seed), "W": make_weight(spec, seed), "bias": make_bias(spec, seed)}


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """View a CPU bf16 tensor as its uint16 bit patterns (no copy)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(a: np.ndarray) -> torch.Tensor:
    """uint16 bit patterns -> CPU bf16 tensor (no copy)."""
    assert a.dtype == np.uint16
    return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
