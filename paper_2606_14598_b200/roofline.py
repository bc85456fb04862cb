"""Work and traffic model of one fused W8A8 linear (no arithmetic of the method itself).

Operation count is 2*M*N*K. The byte model for pre-quantized activations is the
one the paper's roofline classification uses (Results, "compute-bound"
paragraph): int8 activations, int8 weights, 2-byte outputs, scales and bias
ignored. From bf16 activations the quantizer adds a 2-byte read and a 1-byte
write of every activation plus the per-token scales.
"""
from __future__ import annotations

INT8_DENSE_PEAK_TOPS = 4500.0   # B200 datasheet dense INT8 tensor throughput


def ops(M: int, N: int, K: int) -> int:
    return 2 * M * N * K


def bytes_prequantized(M: int, N: int, K: int) -> int:
    return M * K + N * K + 2 * M * N


def quantizer_bytes(M: int, K: int) -> int:
    """bf16 row in, int8 row and one fp32 scale out."""
    return 3 * M * K + 4 * M


def bytes_from_bf16(M: int, N: int, K: int) -> int:
    return quantizer_bytes(M, K) + bytes_prequantized(M, N, K) + 4 * M + 8 * N


def arithmetic_intensity(M: int, N: int, K: int) -> float:
    return ops(M, N, K) / bytes_prequantized(M, N, K)
