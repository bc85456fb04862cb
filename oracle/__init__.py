"""CPU oracle for the fused W8A8 linear layer -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``w8a8_oracle.cpp`` (plain C++, OpenMP over rows).
Only the tests, the smoke check and the benchmark's ``cpu_baseline`` /
``--impl reference`` legs may import this package; the CUDA product never does,
and nothing here imports the product.

All arrays are numpy, C-contiguous unless a leading dimension is given:
bf16 tensors travel as ``uint16`` bit patterns, everything else in its own
dtype. See the header of ``w8a8_oracle.cpp`` for the arithmetic and the
passages of the paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "w8a8_oracle.cpp")
_LIB = os.path.join(_HERE, "libw8a8_oracle.so")
_lock = threading.Lock()
_lib = None

K_MAX = 133144  # largest K with K * 127**2 < 2**31


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no FMA contraction)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".{os.getpid()}.tmp"
            cmd = ["g++", "-std=c++17", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
                   "-shared", "-fPIC", "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i64, vp = ctypes.c_int64, ctypes.c_void_p
        lib.oracle_quantize_weight_per_channel.argtypes = [vp, i64, i64, i64, vp, vp]
        lib.oracle_quantize_weight_per_channel.restype = None
        lib.oracle_quantize_act_per_token.argtypes = [vp, i64, i64, i64, vp, vp]
        lib.oracle_quantize_act_per_token.restype = None
        lib.oracle_quantize_weight_per_channel_smooth.argtypes = [vp, i64, i64, i64, vp, vp, vp]
        lib.oracle_quantize_weight_per_channel_smooth.restype = None
        lib.oracle_quantize_act_per_token_smooth.argtypes = [vp, i64, i64, i64, vp, vp, vp]
        lib.oracle_quantize_act_per_token_smooth.restype = None
        lib.oracle_row_absmax_bf16.argtypes = [vp, i64, i64, i64, vp]
        lib.oracle_row_absmax_bf16.restype = None
        lib.oracle_quantize_act_per_token_given_absmax.argtypes = [vp, i64, i64, i64, vp, vp, vp]
        lib.oracle_quantize_act_per_token_given_absmax.restype = None
        lib.oracle_gemm_i32.argtypes = [vp, vp, vp, i64, i64, i64]
        lib.oracle_gemm_i32.restype = i64
        lib.oracle_epilogue.argtypes = [vp, vp, vp, vp, vp, i64, i64]
        lib.oracle_epilogue.restype = None
        lib.oracle_linear_fused_bf16.argtypes = [vp, i64, vp, vp, vp, vp, i64, i64, i64, vp, vp, vp]
        lib.oracle_linear_fused_bf16.restype = i64
        lib.oracle_num_threads.argtypes = []
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _chk(a, dtype, ndim):
    a = np.asarray(a)
    if a.dtype != dtype or a.ndim != ndim or not a.flags["C_CONTIGUOUS"]:
        raise TypeError(f"expected C-contiguous {dtype} array of rank {ndim}, got {a.dtype} {a.shape}")
    return a


def _chk_rows(a, dtype):
    """Rank-2 array whose rows are contiguous; the rows themselves may be a fixed number of elements apart
    (a column slice of a wider C-contiguous array). Returns (array, row stride in elements)."""
    a = np.asarray(a)
    if a.dtype != dtype or a.ndim != 2:
        raise TypeError(f"expected {dtype} array of rank 2, got {a.dtype} {a.shape}")
    item = a.dtype.itemsize
    if a.shape[1] > 1 and a.strides[1] != item:
        raise TypeError("rows must be contiguous")
    ld = a.strides[0] // item if a.shape[0] > 1 else a.shape[1]
    if a.shape[0] > 1 and (a.strides[0] % item != 0 or ld < a.shape[1]):
        raise TypeError("row stride must be a whole number of elements, at least the row length")
    return a, ld


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def quantize_weight_per_channel(W: np.ndarray):
    """fp32 [N,K] (rows may be strided: a column slice of a wider array) -> (int8 [N,K], fp32 [N])."""
    W, ldw = _chk_rows(W, np.float32)
    N, K = W.shape
    qw = np.empty((N, K), np.int8)
    s_ch = np.empty((N,), np.float32)
    _load().oracle_quantize_weight_per_channel(_p(W), N, K, ldw, _p(qw), _p(s_ch))
    return qw, s_ch


def quantize_act_per_token(A_bits: np.ndarray):
    """bf16 bit patterns uint16 [M,K] (rows may be strided) -> (int8 [M,K], fp32 [M])."""
    A_bits, lda = _chk_rows(A_bits, np.uint16)
    M, K = A_bits.shape
    qa = np.empty((M, K), np.int8)
    s_tok = np.empty((M,), np.float32)
    _load().oracle_quantize_act_per_token(_p(A_bits), M, K, lda, _p(qa), _p(s_tok))
    return qa, s_tok


def row_absmax_bf16(X_bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns uint16 [M,N] (rows may be strided) -> fp32 [M], the largest magnitude of every row."""
    X_bits, ld = _chk_rows(X_bits, np.uint16)
    M, N = X_bits.shape
    rowmax = np.empty((M,), np.float32)
    _load().oracle_row_absmax_bf16(_p(X_bits), M, N, ld, _p(rowmax))
    return rowmax


def quantize_act_per_token_given_absmax(A_bits: np.ndarray, rowmax: np.ndarray):
    """The quantizer's second half: bf16 bit patterns [M,K] and the absmax of every row fp32 [M] -> (int8 [M,K], fp32 [M])."""
    A_bits, lda = _chk_rows(A_bits, np.uint16)
    rowmax = _chk(rowmax, np.float32, 1)
    M, K = A_bits.shape
    assert rowmax.shape == (M,)
    qa = np.empty((M, K), np.int8)
    s_tok = np.empty((M,), np.float32)
    _load().oracle_quantize_act_per_token_given_absmax(_p(A_bits), M, K, lda, _p(rowmax), _p(qa), _p(s_tok))
    return qa, s_tok


def quantize_weight_per_channel_smooth(W: np.ndarray, mult: np.ndarray):
    """fp32 [N,K] times a per-input-channel factor fp32 [K], then quantized per channel."""
    W = _chk(W, np.float32, 2)
    mult = _chk(mult, np.float32, 1)
    N, K = W.shape
    assert mult.shape == (K,)
    qw = np.empty((N, K), np.int8)
    s_ch = np.empty((N,), np.float32)
    _load().oracle_quantize_weight_per_channel_smooth(_p(W), N, K, K, _p(mult), _p(qw), _p(s_ch))
    return qw, s_ch


def quantize_act_per_token_smooth(A_bits: np.ndarray, mult: np.ndarray):
    """bf16 bit patterns [M,K] times a per-input-channel factor fp32 [K], then quantized per token."""
    A_bits = _chk(A_bits, np.uint16, 2)
    mult = _chk(mult, np.float32, 1)
    M, K = A_bits.shape
    assert mult.shape == (K,)
    qa = np.empty((M, K), np.int8)
    s_tok = np.empty((M,), np.float32)
    _load().oracle_quantize_act_per_token_smooth(_p(A_bits), M, K, K, _p(mult), _p(qa), _p(s_tok))
    return qa, s_tok


def linear_fused_bf16_smooth(A_bits, a_mult, qw, s_ch, bias):
    """Whole path from bf16 activations smoothed by a_mult. Returns dict(out, qa, s_tok, acc)."""
    qa, s_tok = quantize_act_per_token_smooth(A_bits, a_mult)
    r = linear_fused_int8(qa, s_tok, qw, s_ch, bias)
    r.update(qa=qa, s_tok=s_tok)
    return r


def gemm_i32(qa: np.ndarray, qw: np.ndarray) -> np.ndarray:
    """int8 [M,K] x int8 [N,K]^T -> int32 [M,N]; raises if any sum leaves int32."""
    qa = _chk(qa, np.int8, 2)
    qw = _chk(qw, np.int8, 2)
    M, K = qa.shape
    N, K2 = qw.shape
    if K != K2:
        raise ValueError("K mismatch")
    acc = np.empty((M, N), np.int32)
    bad = _load().oracle_gemm_i32(_p(qa), _p(qw), _p(acc), M, N, K)
    if bad:
        raise OverflowError(f"{bad} accumulators do not fit in int32")
    return acc


def epilogue(acc: np.ndarray, s_tok: np.ndarray, s_ch: np.ndarray, bias: np.ndarray | None) -> np.ndarray:
    """int32 [M,N], fp32 [M], fp32 [N], fp32 [N] or None -> bf16 bit patterns uint16 [M,N]."""
    acc = _chk(acc, np.int32, 2)
    M, N = acc.shape
    s_tok = _chk(s_tok, np.float32, 1)
    s_ch = _chk(s_ch, np.float32, 1)
    if bias is not None:
        bias = _chk(bias, np.float32, 1)
        assert bias.shape == (N,)
    assert s_tok.shape == (M,) and s_ch.shape == (N,)
    out = np.empty((M, N), np.uint16)
    _load().oracle_epilogue(_p(acc), _p(s_tok), _p(s_ch), _p(bias), _p(out), M, N)
    return out


def linear_fused_bf16(A_bits, qw, s_ch, bias):
    """Whole path from bf16 activations. Returns dict(out, qa, s_tok, acc)."""
    A_bits = _chk(A_bits, np.uint16, 2)
    qw = _chk(qw, np.int8, 2)
    M, K = A_bits.shape
    N = qw.shape[0]
    assert qw.shape[1] == K
    s_ch = _chk(s_ch, np.float32, 1)
    if bias is not None:
        bias = _chk(bias, np.float32, 1)
    qa = np.empty((M, K), np.int8)
    s_tok = np.empty((M,), np.float32)
    acc = np.empty((M, N), np.int32)
    out = np.empty((M, N), np.uint16)
    bad = _load().oracle_linear_fused_bf16(_p(A_bits), K, _p(qw), _p(s_ch), _p(bias), _p(out),
                                           M, N, K, _p(qa), _p(s_tok), _p(acc))
    if bad:
        raise OverflowError(f"{bad} accumulators do not fit in int32")
    return {"out": out, "qa": qa, "s_tok": s_tok, "acc": acc}


def linear_fused_int8(qa, s_tok, qw, s_ch, bias):
    """Whole path from pre-quantized activations. Returns dict(out, acc)."""
    acc = gemm_i32(qa, qw)
    return {"out": epilogue(acc, s_tok, s_ch, bias), "acc": acc}
