"""ctypes binding of libw8a8_linear.so: the same entry points as include/w8a8_linear.h.

Marshalling only: tensors are allocated with torch (device memory, streams),
their pointers and sizes are handed to the C ABI, and every step of the path
runs inside the library's CUDA kernels. There is no fallback: if the shared
library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libw8a8_linear.so")

ACT_BF16 = 0
ACT_INT8 = 1
K_MAX = 133144

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "ALIGNMENT", 3: "K_OVERFLOW", 4: "WORKSPACE", 5: "ARCH", 6: "CUDA", 7: "TIMEOUT"}

EXPORTS = (
    "int8_quantize_weight_per_channel", "int8_quantize_act_per_token", "int8_linear_workspace_bytes",
    "int8_linear_workspace_offsets", "int8_linear_fused", "int8_linear_fused_host", "int8_gemm_i32_debug",
    "int8_check_status", "int8_linear_force_config", "int8_linear_num_configs", "int8_linear_config_name",
    "int8_status_string", "int8_linear_fused_static", "int8_quantize_weight_per_channel_smooth",
    "int8_quantize_act_per_token_smooth", "int8_linear_fused_smooth", "int8_linear_workspace_min_bytes", "int8_linear_plan",
    "int8_sticky_status", "int8_debug_set_wait_limit_ns", "int8_debug_set_starve", "int8_debug_set_small_path",
    "int8_linear_fused_rowmax", "int8_quantize_act_per_token_given_absmax", "int8_linear_fused_given_absmax",
)

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it first (python -c 'import __graft_entry__ as g; g.build()'). "
        "This package has no CPU or PyTorch fallback.")

_lib = ctypes.CDLL(LIB_PATH)
_i64, _vp, _sz, _int = ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int

_lib.int8_quantize_weight_per_channel.argtypes = [_vp, _i64, _i64, _i64, _vp, _vp, _vp]
_lib.int8_quantize_weight_per_channel.restype = _int
_lib.int8_quantize_act_per_token.argtypes = [_vp, _i64, _i64, _i64, _vp, _vp, _vp]
_lib.int8_quantize_act_per_token.restype = _int
_lib.int8_linear_workspace_bytes.argtypes = [_i64, _i64, _i64, _int]
_lib.int8_linear_workspace_bytes.restype = _sz
_lib.int8_linear_workspace_min_bytes.argtypes = [_i64, _i64, _i64, _int]
_lib.int8_linear_workspace_min_bytes.restype = _sz
_lib.int8_linear_plan.argtypes = [_i64, _i64, _i64, _int, _sz] + [ctypes.POINTER(_int)] * 4
_lib.int8_linear_plan.restype = _int
_lib.int8_linear_workspace_offsets.argtypes = [_i64, _i64, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]
_lib.int8_linear_workspace_offsets.restype = None
_lib.int8_linear_fused.argtypes = [_vp, _int, _i64, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i64, _vp, _sz, _vp]
_lib.int8_linear_fused.restype = _int
_lib.int8_linear_fused_host.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _sz, _vp]
_lib.int8_linear_fused_host.restype = _int
_lib.int8_linear_fused_static.argtypes = [_vp, _i64, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i64, _int, _vp]
_lib.int8_linear_fused_static.restype = _int
_lib.int8_quantize_weight_per_channel_smooth.argtypes = [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp]
_lib.int8_quantize_weight_per_channel_smooth.restype = _int
_lib.int8_quantize_act_per_token_smooth.argtypes = [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp]
_lib.int8_quantize_act_per_token_smooth.restype = _int
_lib.int8_linear_fused_smooth.argtypes = [_vp, _i64, _vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i64, _vp, _sz, _vp]
_lib.int8_linear_fused_smooth.restype = _int
_lib.int8_linear_fused_rowmax.argtypes = [_vp, _int, _i64, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _i64, _i64, _i64, _vp, _sz, _vp]
_lib.int8_linear_fused_rowmax.restype = _int
_lib.int8_quantize_act_per_token_given_absmax.argtypes = [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _vp]
_lib.int8_quantize_act_per_token_given_absmax.restype = _int
_lib.int8_linear_fused_given_absmax.argtypes = [_vp, _i64, _vp, _vp, _vp, _vp, _vp, _i64, _vp, _i64, _i64, _i64, _vp, _sz, _vp]
_lib.int8_linear_fused_given_absmax.restype = _int
_lib.int8_gemm_i32_debug.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _vp, _sz, _vp]
_lib.int8_gemm_i32_debug.restype = _int
_lib.int8_check_status.argtypes = [_vp, _vp]
_lib.int8_check_status.restype = _int
_lib.int8_sticky_status.argtypes = [_int, _vp]
_lib.int8_sticky_status.restype = _int
_lib.int8_debug_set_wait_limit_ns.argtypes = [ctypes.c_uint64]
_lib.int8_debug_set_wait_limit_ns.restype = ctypes.c_uint64
_lib.int8_debug_set_starve.argtypes = [_int]
_lib.int8_debug_set_starve.restype = _int
_lib.int8_debug_set_small_path.argtypes = [_int]
_lib.int8_debug_set_small_path.restype = _int
_lib.int8_linear_force_config.argtypes = [_int]
_lib.int8_linear_force_config.restype = _int
_lib.int8_linear_num_configs.argtypes = []
_lib.int8_linear_num_configs.restype = _int
_lib.int8_linear_config_name.argtypes = [_int]
_lib.int8_linear_config_name.restype = ctypes.c_char_p
_lib.int8_status_string.argtypes = [_int]
_lib.int8_status_string.restype = ctypes.c_char_p


class W8A8Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.int8_status_string(status).decode()
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({msg})")


def raw():
    """The ctypes library object (for tests that call the C ABI with hand-made arguments)."""
    return _lib


def _check(status: int, where: str):
    if status != 0:
        raise W8A8Error(status, where)


def _ptr(t: torch.Tensor | None):
    return None if t is None else t.data_ptr()


def _stream(t: torch.Tensor):
    return torch.cuda.current_stream(t.device).cuda_stream if t.is_cuda else None


def _need(t: torch.Tensor, dtype, name: str, ndim: int):
    if t.dtype != dtype or t.dim() != ndim:
        raise TypeError(f"{name}: expected {dtype} tensor of rank {ndim}, got {t.dtype} {tuple(t.shape)}")
    if ndim == 2 and t.stride(1) != 1:
        raise TypeError(f"{name}: rows must be contiguous")
    if ndim == 1 and t.numel() > 1 and t.stride(0) != 1:
        raise TypeError(f"{name}: must be contiguous")


def status_string(status: int) -> str:
    return _lib.int8_status_string(status).decode()


def force_config(config_id: int) -> int:
    return _lib.int8_linear_force_config(config_id)


def num_configs() -> int:
    return _lib.int8_linear_num_configs()


def config_name(config_id: int) -> str | None:
    s = _lib.int8_linear_config_name(config_id)
    return None if s is None else s.decode()


def int8_quantize_weight_per_channel(W: torch.Tensor):
    """fp32 [N,K] device tensor -> (int8 [N,K], fp32 [N])."""
    _need(W, torch.float32, "W", 2)
    N, K = W.shape
    qw = torch.empty((N, K), dtype=torch.int8, device=W.device)
    s_ch = torch.empty((N,), dtype=torch.float32, device=W.device)
    _check(_lib.int8_quantize_weight_per_channel(_ptr(W), N, K, W.stride(0), _ptr(qw), _ptr(s_ch), _stream(W)),
           "int8_quantize_weight_per_channel")
    return qw, s_ch


def int8_quantize_act_per_token(A: torch.Tensor, qa: torch.Tensor | None = None, s_tok: torch.Tensor | None = None):
    """bf16 [M,K] device tensor -> (int8 [M,K], fp32 [M])."""
    _need(A, torch.bfloat16, "A", 2)
    M, K = A.shape
    if qa is None:
        qa = torch.empty((M, K), dtype=torch.int8, device=A.device)
    if s_tok is None:
        s_tok = torch.empty((M,), dtype=torch.float32, device=A.device)
    _check(_lib.int8_quantize_act_per_token(_ptr(A), M, K, A.stride(0), _ptr(qa), _ptr(s_tok), _stream(A)),
           "int8_quantize_act_per_token")
    return qa, s_tok


def int8_quantize_weight_per_channel_smooth(W: torch.Tensor, w_mult: torch.Tensor):
    """fp32 [N,K] times the per-input-channel factors fp32 [K] (SmoothQuant hook) -> (int8 [N,K], fp32 [N])."""
    _need(W, torch.float32, "W", 2)
    _need(w_mult, torch.float32, "w_mult", 1)
    N, K = W.shape
    if w_mult.shape[0] != K:
        raise ValueError("w_mult must have K entries")
    qw = torch.empty((N, K), dtype=torch.int8, device=W.device)
    s_ch = torch.empty((N,), dtype=torch.float32, device=W.device)
    _check(_lib.int8_quantize_weight_per_channel_smooth(_ptr(W), N, K, W.stride(0), _ptr(w_mult), _ptr(qw), _ptr(s_ch),
                                                        _stream(W)), "int8_quantize_weight_per_channel_smooth")
    return qw, s_ch


def int8_quantize_act_per_token_smooth(A: torch.Tensor, a_mult: torch.Tensor):
    """bf16 [M,K] times the per-input-channel factors fp32 [K] (SmoothQuant hook) -> (int8 [M,K], fp32 [M])."""
    _need(A, torch.bfloat16, "A", 2)
    _need(a_mult, torch.float32, "a_mult", 1)
    M, K = A.shape
    if a_mult.shape[0] != K:
        raise ValueError("a_mult must have K entries")
    qa = torch.empty((M, K), dtype=torch.int8, device=A.device)
    s_tok = torch.empty((M,), dtype=torch.float32, device=A.device)
    _check(_lib.int8_quantize_act_per_token_smooth(_ptr(A), M, K, A.stride(0), _ptr(a_mult), _ptr(qa), _ptr(s_tok),
                                                   _stream(A)), "int8_quantize_act_per_token_smooth")
    return qa, s_tok


def int8_linear_fused_smooth(A: torch.Tensor, a_mult: torch.Tensor, qw: torch.Tensor, s_ch: torch.Tensor,
                             bias: torch.Tensor | None = None, out: torch.Tensor | None = None,
                             workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Fused linear on bf16 activations smoothed by a_mult (weights quantized with the matching w_mult)."""
    _need(A, torch.bfloat16, "A", 2)
    _need(a_mult, torch.float32, "a_mult", 1)
    _need(qw, torch.int8, "qw", 2)
    _need(s_ch, torch.float32, "s_ch", 1)
    M, K = A.shape
    N = qw.shape[0]
    if qw.shape[1] != K or s_ch.shape[0] != N or a_mult.shape[0] != K or not qw.is_contiguous():
        raise ValueError("shape mismatch")
    if bias is not None:
        _need(bias, torch.float32, "bias", 1)
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, ACT_BF16, A.device)
    _check(_lib.int8_linear_fused_smooth(_ptr(A), A.stride(0), _ptr(a_mult), _ptr(qw), _ptr(s_ch), _ptr(bias), _ptr(out),
                                         out.stride(0), M, N, K, _ptr(workspace), workspace.numel(), _stream(A)),
           "int8_linear_fused_smooth")
    return out


def int8_quantize_act_per_token_given_absmax(A: torch.Tensor, rowmax: torch.Tensor):
    """One-pass quantizer: bf16 [M,K] and the absmax of every row fp32 [M] (>= the true one) -> (int8 [M,K], fp32 [M])."""
    _need(A, torch.bfloat16, "A", 2)
    _need(rowmax, torch.float32, "rowmax", 1)
    M, K = A.shape
    if rowmax.shape[0] != M:
        raise ValueError("rowmax must have M entries")
    qa = torch.empty((M, K), dtype=torch.int8, device=A.device)
    s_tok = torch.empty((M,), dtype=torch.float32, device=A.device)
    _check(_lib.int8_quantize_act_per_token_given_absmax(_ptr(A), M, K, A.stride(0), _ptr(rowmax), _ptr(qa), _ptr(s_tok),
                                                         _stream(A)), "int8_quantize_act_per_token_given_absmax")
    return qa, s_tok


def int8_linear_fused_rowmax(A: torch.Tensor, qw: torch.Tensor, s_ch: torch.Tensor, bias: torch.Tensor | None = None,
                             s_tok: torch.Tensor | None = None, out: torch.Tensor | None = None,
                             workspace: torch.Tensor | None = None, rowmax_in: torch.Tensor | None = None):
    """Fused linear that also returns rowmax[m] = max_n |out[m,n]| (fp32 [M]). With rowmax_in (bf16 activations only)
    the quantizer runs in one pass on the absmax handed in. Returns (out, rowmax)."""
    a_dtype = ACT_BF16 if A.dtype == torch.bfloat16 else ACT_INT8
    _need(A, torch.bfloat16 if a_dtype == ACT_BF16 else torch.int8, "A", 2)
    _need(qw, torch.int8, "qw", 2)
    _need(s_ch, torch.float32, "s_ch", 1)
    M, K = A.shape
    N = qw.shape[0]
    if qw.shape[1] != K or s_ch.shape[0] != N or not qw.is_contiguous():
        raise ValueError("shape mismatch")
    if bias is not None:
        _need(bias, torch.float32, "bias", 1)
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, a_dtype, A.device)
    rowmax = torch.empty((M,), dtype=torch.float32, device=A.device)
    if rowmax_in is None:
        _check(_lib.int8_linear_fused_rowmax(_ptr(A), a_dtype, A.stride(0), _ptr(s_tok), _ptr(qw), _ptr(s_ch), _ptr(bias),
                                             _ptr(out), out.stride(0), _ptr(rowmax), M, N, K, _ptr(workspace),
                                             workspace.numel(), _stream(A)), "int8_linear_fused_rowmax")
    else:
        _need(rowmax_in, torch.float32, "rowmax_in", 1)
        if a_dtype != ACT_BF16 or rowmax_in.shape[0] != M:
            raise ValueError("rowmax_in goes with bf16 activations and has M entries")
        _check(_lib.int8_linear_fused_given_absmax(_ptr(A), A.stride(0), _ptr(rowmax_in), _ptr(qw), _ptr(s_ch), _ptr(bias),
                                                   _ptr(out), out.stride(0), _ptr(rowmax), M, N, K, _ptr(workspace),
                                                   workspace.numel(), _stream(A)), "int8_linear_fused_given_absmax")
    return out, rowmax


def int8_linear_workspace_bytes(M: int, N: int, K: int, a_dtype: int = ACT_BF16) -> int:
    return int(_lib.int8_linear_workspace_bytes(M, N, K, a_dtype))


def int8_linear_workspace_min_bytes(M: int, N: int, K: int, a_dtype: int = ACT_BF16) -> int:
    return int(_lib.int8_linear_workspace_min_bytes(M, N, K, a_dtype))


def int8_linear_plan(M: int, N: int, K: int, a_dtype: int = ACT_BF16, workspace_bytes: int | None = None) -> dict:
    """How the fused call would run this shape: {'config', 'name', 'groups', 'split_tiles', 'split_parts'}."""
    if workspace_bytes is None:
        workspace_bytes = int8_linear_workspace_bytes(M, N, K, a_dtype)
    v = [_int(0) for _ in range(4)]
    _check(_lib.int8_linear_plan(M, N, K, a_dtype, workspace_bytes, *[ctypes.byref(x) for x in v]), "int8_linear_plan")
    cfg = int(v[0].value)
    return {"config": cfg, "name": config_name(cfg), "groups": int(v[1].value),
            "split_tiles": int(v[2].value), "split_parts": int(v[3].value)}


def int8_linear_workspace_offsets(M: int, K: int):
    a, b = _sz(0), _sz(0)
    _lib.int8_linear_workspace_offsets(M, K, ctypes.byref(a), ctypes.byref(b))
    return int(a.value), int(b.value)


def alloc_workspace(M: int, N: int, K: int, a_dtype: int = ACT_BF16, device="cuda") -> torch.Tensor:
    """Device scratch for int8_linear_fused (torch caching-allocator blocks are 512-byte aligned)."""
    return torch.empty((int8_linear_workspace_bytes(M, N, K, a_dtype),), dtype=torch.uint8, device=device)


def int8_linear_fused(A: torch.Tensor, qw: torch.Tensor, s_ch: torch.Tensor, bias: torch.Tensor | None = None,
                      s_tok: torch.Tensor | None = None, out: torch.Tensor | None = None,
                      workspace: torch.Tensor | None = None) -> torch.Tensor:
    """out[M,N] bf16 = dequant(quant(A) @ qw^T) + bias. A is bf16 [M,K], or int8 [M,K] with s_tok fp32 [M]."""
    if A.dtype == torch.bfloat16:
        a_dtype = ACT_BF16
    elif A.dtype == torch.int8:
        a_dtype = ACT_INT8
    else:
        raise TypeError(f"A: bf16 or int8 expected, got {A.dtype}")
    _need(A, A.dtype, "A", 2)
    _need(qw, torch.int8, "qw", 2)
    _need(s_ch, torch.float32, "s_ch", 1)
    if not qw.is_contiguous():
        raise TypeError("qw must be dense")
    M, K = A.shape
    N = qw.shape[0]
    if qw.shape[1] != K or s_ch.shape[0] != N:
        raise ValueError("shape mismatch")
    if bias is not None:
        _need(bias, torch.float32, "bias", 1)
    if s_tok is not None:
        _need(s_tok, torch.float32, "s_tok", 1)
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)
    _need(out, torch.bfloat16, "out", 2)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, a_dtype, A.device)
    _check(_lib.int8_linear_fused(_ptr(A), a_dtype, A.stride(0), _ptr(s_tok), _ptr(qw), _ptr(s_ch), _ptr(bias),
                                  _ptr(out), out.stride(0), M, N, K, _ptr(workspace), workspace.numel(), _stream(A)),
           "int8_linear_fused")
    return out


def int8_linear_fused_host(A_host: torch.Tensor, d_A: torch.Tensor, qw: torch.Tensor, s_ch: torch.Tensor,
                           bias: torch.Tensor | None, d_out: torch.Tensor, out_host: torch.Tensor,
                           workspace: torch.Tensor) -> torch.Tensor:
    """Host-buffer variant: A_host/out_host are (pinned) CPU bf16 tensors, the rest device tensors."""
    M, K = A_host.shape
    N = qw.shape[0]
    assert not A_host.is_cuda and not out_host.is_cuda and d_A.is_cuda and d_out.is_cuda
    assert A_host.is_contiguous() and out_host.is_contiguous() and d_A.is_contiguous() and d_out.is_contiguous()
    _check(_lib.int8_linear_fused_host(_ptr(A_host), _ptr(d_A), _ptr(qw), _ptr(s_ch), _ptr(bias), _ptr(d_out),
                                       _ptr(out_host), M, N, K, _ptr(workspace), workspace.numel(), _stream(d_A)),
           "int8_linear_fused_host")
    return out_host


STATIC_WORKSPACE_BYTES = 16 * 1024 * 1024


def int8_linear_fused_static(A: torch.Tensor, qw: torch.Tensor, s_ch: torch.Tensor, bias: torch.Tensor | None = None,
                             out: torch.Tensor | None = None, sync_and_check: bool = False) -> torch.Tensor:
    """Fused linear on bf16 activations whose scratch is the library's built-in device array: no workspace
    argument and no allocation inside the call. For callers that cannot allocate (see the header). Refuses
    problems whose scratch exceeds STATIC_WORKSPACE_BYTES; calls that overlap on the GPU share the array and race."""
    _need(A, torch.bfloat16, "A", 2)
    _need(qw, torch.int8, "qw", 2)
    _need(s_ch, torch.float32, "s_ch", 1)
    M, K = A.shape
    N = qw.shape[0]
    if qw.shape[1] != K or s_ch.shape[0] != N or not qw.is_contiguous():
        raise ValueError("shape mismatch")
    if bias is not None:
        _need(bias, torch.float32, "bias", 1)
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=A.device)   # the caller's output, not scratch
    _need(out, torch.bfloat16, "out", 2)
    _check(_lib.int8_linear_fused_static(_ptr(A), A.stride(0), _ptr(qw), _ptr(s_ch), _ptr(bias), _ptr(out),
                                         out.stride(0), M, N, K, 1 if sync_and_check else 0, _stream(A)),
           "int8_linear_fused_static")
    return out


def int8_gemm_i32_debug(qa: torch.Tensor, qw: torch.Tensor, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """Raw int32 accumulators of the GEMM path (test-only export)."""
    _need(qa, torch.int8, "qa", 2)
    _need(qw, torch.int8, "qw", 2)
    M, K = qa.shape
    N = qw.shape[0]
    acc = torch.empty((M, N), dtype=torch.int32, device=qa.device)
    if workspace is None:
        workspace = alloc_workspace(M, N, K, ACT_INT8, qa.device)
    _check(_lib.int8_gemm_i32_debug(_ptr(qa.contiguous()), _ptr(qw.contiguous()), _ptr(acc), M, N, K,
                                    _ptr(workspace), workspace.numel(), _stream(qa)), "int8_gemm_i32_debug")
    return acc


def int8_sticky_status(clear: bool = True, device=None) -> int:
    """First time-out recorded by any call on the current device since the last clear (synchronizes the current stream)."""
    stream = torch.cuda.current_stream(device).cuda_stream
    return int(_lib.int8_sticky_status(1 if clear else 0, stream))


def debug_set_wait_limit_ns(limit_ns: int) -> int:
    """Test-only: bound of the device-side waits of the following launches (0 = the 2 s default). Returns the old value."""
    return int(_lib.int8_debug_set_wait_limit_ns(int(limit_ns)))


def debug_set_starve(mode: int) -> int:
    """Test-only: 1 = the GEMM's producer withholds a stage, 2 = the quantizer's producer does; 0 = off."""
    return int(_lib.int8_debug_set_starve(int(mode)))


def debug_set_small_path(mode: int) -> int:
    """Test-only: -1 = the one-kernel path where the shape calls for it (default), 0 = never, 1 = wherever it can run."""
    return int(_lib.int8_debug_set_small_path(int(mode)))


def gemm_clock_stamps(workspace: torch.Tensor):
    """(SM clock in MHz, seconds) of the first CTA of the last tensor-core GEMM that ran on this workspace, from the
    diagnostics stamps in the status block; None if no such launch has left stamps. Synchronizes (copies to the host)."""
    c0, t0, c1, t1 = workspace[64:96].view(torch.int64).tolist()
    if t1 <= t0 or c1 <= c0:
        return None
    return (c1 - c0) / (t1 - t0) * 1e3, (t1 - t0) * 1e-9


def int8_check_status(workspace: torch.Tensor) -> int:
    """Synchronizes the current stream and returns (then clears) the workspace's device-side status."""
    return int(_lib.int8_check_status(_ptr(workspace), _stream(workspace)))
