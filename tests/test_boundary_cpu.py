"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, sizes workspaces as documented, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

import paper_2606_14598_b200 as w8
from paper_2606_14598_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "w8a8_linear.h")


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(int8_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert len(names) >= 10
    lib = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_status_strings():
    for code in range(8):
        assert w8.status_string(code) and w8.status_string(code) != "unknown status"
    assert w8.status_string(99) == "unknown status"


def test_workspace_sizes():
    assert w8.int8_linear_workspace_bytes(4608, 3072, 12288, w8.ACT_INT8) == 256
    # status block, s_tok (padded to 256), qa
    s_off, q_off = w8.int8_linear_workspace_offsets(4608, 12288)
    assert s_off == 256 and q_off == s_off + 4608 * 4 and q_off % 256 == 0
    assert w8.int8_linear_workspace_bytes(4608, 3072, 12288, w8.ACT_BF16) == q_off + 4608 * 12288
    s_off, q_off = w8.int8_linear_workspace_offsets(2, 3072)
    assert s_off == 256 and q_off == 512 and w8.int8_linear_workspace_bytes(2, 8, 3072, w8.ACT_BF16) == 512 + 6144
    assert w8.int8_linear_workspace_bytes(0, 8, 16) == 0
    assert w8.int8_linear_workspace_bytes(8, 8, 16, 5) == 0
    # the smallest accepted workspace is the layout above; the recommended one adds room for the partial sums of
    # the K-split where the shape's last wave of tiles is mostly empty and K is deep (the paper's llm-proj), and
    # nothing where it is not (the c4 shapes) or where the CUDA-core path runs (M <= 8)
    for (M, N, K) in [(4608, 3072, 12288), (4608, 12288, 3072), (4110, 4608, 53248), (512, 4608, 53248), (2, 18432, 3072)]:
        for dt in (w8.ACT_BF16, w8.ACT_INT8):
            lo, hi = w8.int8_linear_workspace_min_bytes(M, N, K, dt), w8.int8_linear_workspace_bytes(M, N, K, dt)
            assert lo % 256 == 0 and hi % 256 == 0 and lo <= hi <= lo + (12 << 20)
            if dt == w8.ACT_BF16:
                assert lo == w8.int8_linear_workspace_offsets(M, K)[1] + (M * K + 255) // 256 * 256
            else:
                assert lo == 256
            assert (hi > lo) == (K == 53248), (M, N, K, lo, hi)


def test_plan_of_the_benchmark_shapes():
    # the static per-shape choice (148 SMs assumed without a device): CTA pairs with 256x256 tiles on the large
    # shapes; deep K with a nearly empty last wave is cut along K when the workspace has room, and only then.
    # From three waves of tiles on, the grid is the fewest pairs that need no more waves (216 tiles: 72 pairs x 3).
    w8.force_config(-1)
    pair = next(i for i in range(w8.num_configs()) if "256x256 per CTA pair" in w8.config_name(i))
    for (M, N, K, groups) in [(4608, 12288, 3072, 72), (4608, 3072, 12288, 72), (9216, 9216, 3072, 72), (2816, 3072, 3072, 74)]:
        p = w8.int8_linear_plan(M, N, K, w8.ACT_BF16)
        assert p["config"] == pair and p["split_parts"] == 0 and p["groups"] == groups, p
    p = w8.int8_linear_plan(4110, 4608, 53248, w8.ACT_BF16)
    assert p["config"] == pair and p["groups"] == 74 and p["split_tiles"] == 306 % 74 and p["split_parts"] == 7, p
    lo = w8.int8_linear_workspace_min_bytes(4110, 4608, 53248, w8.ACT_BF16)
    assert w8.int8_linear_plan(4110, 4608, 53248, w8.ACT_BF16, lo)["split_parts"] == 0
    p = w8.int8_linear_plan(512, 4608, 53248, w8.ACT_INT8)
    assert p["split_parts"] == 2 and p["groups"] == p["split_tiles"] * 2 <= 74, p
    assert w8.int8_linear_plan(4110, 4608, 4608, w8.ACT_BF16)["split_parts"] == 0       # shallow K: a cut would not pay
    assert w8.int8_linear_plan(2, 18432, 3072, w8.ACT_BF16)["config"] == w8.num_configs() - 1   # CUDA-core path
    assert "128x128" in w8.int8_linear_plan(128, 256, 256, w8.ACT_INT8)["name"] or \
           "256x128" in w8.int8_linear_plan(128, 256, 256, w8.ACT_INT8)["name"]
    # forcing a configuration cuts whenever it can; + 0x100 never cuts; -2 chooses freely but never cuts
    w8.force_config(pair)
    assert w8.int8_linear_plan(256, 512, 2048, w8.ACT_INT8, 64 << 20)["split_parts"] == 2
    w8.force_config(pair + 0x100)
    assert w8.int8_linear_plan(256, 512, 2048, w8.ACT_INT8, 64 << 20)["split_parts"] == 0
    w8.force_config(-2)
    assert w8.int8_linear_plan(4110, 4608, 53248, w8.ACT_BF16)["split_parts"] == 0
    w8.force_config(-1)
    with pytest.raises(w8.W8A8Error):
        w8.int8_linear_plan(4110, 4608, 53248, w8.ACT_BF16, 1024)                       # below the minimum


def test_one_kernel_path_is_chosen_for_one_tile_problems_only():
    """Host logic of the default mode: problems of a few dozen tokens and a small A take the one-kernel path; larger
    or skinnier problems, forced configurations and pre-quantized activations do not."""
    ws_big = 1 << 30
    name = lambda M, N, K, a=w8.ACT_BF16: w8.int8_linear_plan(M, N, K, a, ws_big)["name"]
    assert "one kernel" in name(64, 512, 512)
    assert "one kernel" in name(16, 1024, 512)
    assert "one kernel" in name(16, 64, 1024)           # N = 64: a cluster of two shares 16 Ki elements
    assert "one kernel" not in name(32, 64, 1024)       # ... but not 32 Ki
    assert "one kernel" not in name(64, 512, 512, w8.ACT_INT8)
    assert "one kernel" not in name(64, 1024, 1024)     # 16 Ki elements per CTA of a cluster of four
    assert "one kernel" not in name(128, 256, 256)      # c1: more than 64 tokens
    assert "one kernel" not in name(64, 2048, 256)      # N > 1024
    assert "one kernel" not in name(8, 256, 256)        # skinny: the weight-streaming kernel
    assert "one kernel" not in name(2816, 3072, 3072)
    w8.force_config(0)
    try:
        assert "one kernel" not in name(64, 512, 512)
    finally:
        w8.force_config(-1)


def test_configs_are_listed():
    n = w8.num_configs()
    # ids below n can be forced; id n only appears in plans (the one-kernel path for small problems is chosen by shape)
    assert n >= 2 and all(w8.config_name(i) for i in range(n)) and "one kernel" in w8.config_name(n)
    assert w8.config_name(n + 1) is None
    assert w8.force_config(-1) == -1


# fake, well-aligned addresses: argument checks run before any CUDA call, so nothing is dereferenced
P = 0x10000


def fused(A=P, a_dtype=0, lda=64, s_tok=None, qw=P, s_ch=P, bias=None, out=P, ldo=64, M=32, N=64, K=64, ws=P, ws_bytes=1 << 20):
    return binding.raw().int8_linear_fused(A, a_dtype, lda, s_tok, qw, s_ch, bias, out, ldo, M, N, K, ws, ws_bytes, None)


def test_fused_rejects_bad_arguments_before_any_launch():
    INVALID, ALIGN, KOVF, WS = 1, 2, 3, 4
    assert fused(A=None) == INVALID
    assert fused(qw=None) == INVALID and fused(s_ch=None) == INVALID and fused(out=None) == INVALID
    assert fused(a_dtype=2) == INVALID
    assert fused(a_dtype=1, s_tok=None) == INVALID          # int8 activations need their scales
    assert fused(a_dtype=0, s_tok=P) == INVALID             # bf16 activations must not bring scales
    assert fused(M=0) == INVALID and fused(N=-8) == INVALID and fused(K=0) == INVALID
    assert fused(lda=32) == INVALID and fused(ldo=56) == INVALID
    assert fused(K=133152, lda=133152) == KOVF
    assert fused(K=w8.K_MAX + 8, lda=w8.K_MAX + 8) == KOVF
    assert fused(K=72, lda=72) == ALIGN                     # K % 16
    assert fused(N=60, ldo=64) == ALIGN                     # N % 8
    assert fused(ldo=68) == ALIGN
    assert fused(a_dtype=1, s_tok=P, lda=72) == ALIGN       # int8 row stride not a multiple of 16 bytes
    assert fused(A=P + 8) == ALIGN and fused(qw=P + 4) == ALIGN and fused(out=P + 2) == ALIGN
    assert fused(ws=None) == WS and fused(ws=P + 128) == WS and fused(ws_bytes=255) == WS
    need = w8.int8_linear_workspace_min_bytes(32, 64, 64, 0)
    assert fused(ws_bytes=need - 1) == WS


def test_quantizers_reject_bad_arguments():
    lib = binding.raw()
    assert lib.int8_quantize_weight_per_channel(None, 8, 16, 16, P, P, None) == 1
    assert lib.int8_quantize_weight_per_channel(P, 8, 16, 8, P, P, None) == 1      # ldw < K
    assert lib.int8_quantize_weight_per_channel(P, 8, 24, 24, P, P, None) == 2     # K % 16
    assert lib.int8_quantize_weight_per_channel(P + 4, 8, 16, 16, P, P, None) == 2
    assert lib.int8_quantize_act_per_token(P, 0, 16, 16, P, P, None) == 1
    assert lib.int8_quantize_act_per_token(P, 8, 16, 20, P, P, None) == 2          # lda % 8
    assert lib.int8_gemm_i32_debug(P, P, None, 8, 8, 16, P, 256, None) == 1
    assert lib.int8_gemm_i32_debug(P, P, P, 8, 6, 16, P, 256, None) == 2
    assert lib.int8_gemm_i32_debug(P, P, P, 8, 8, 16, P, 8, None) == 4
    assert lib.int8_check_status(None, None) == 4
    # SmoothQuant entry points: the factor vector is required and must be 16-byte aligned
    assert lib.int8_quantize_weight_per_channel_smooth(P, 8, 16, 16, None, P, P, None) == 1
    assert lib.int8_quantize_act_per_token_smooth(P, 8, 16, 16, P + 4, P, P, None) == 2
    assert lib.int8_linear_fused_smooth(P, 64, None, P, P, None, P, 64, 32, 64, 64, P, 1 << 20, None) == 1


def test_no_device_means_a_loud_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    # valid arguments, no device: the call must fail (CUDA error), never compute on the CPU
    assert fused() in (5, 6)


def test_oracle_side_processes_do_not_map_the_cuda_library():
    # The generator, the work model, the multi-rank plumbing and the oracle must run in a process that never
    # maps libw8a8_linear.so (the oracle's independence is only worth something if its processes are free of
    # the product); the library is loaded by the first touch of a compute entry point, and only then.
    import subprocess
    import sys
    import textwrap
    code = textwrap.dedent("""
        import sys
        sys.path.insert(0, %r)
        import numpy as np
        import oracle
        import paper_2606_14598_b200 as pkg
        from paper_2606_14598_b200 import inputs, roofline, dist
        t = inputs.make_linear(inputs.LinearSpec("indep", 8, 32, 16))
        qw, s_ch = oracle.quantize_weight_per_channel(t["W"].numpy())
        out = oracle.linear_fused_bf16(inputs.bf16_bits(t["A"]), qw, s_ch, t["bias"].numpy())["out"]
        assert out.shape == (8, 16) and roofline.ops(8, 16, 32) == 8192 and dist.shard_rows(8, 0, 2) == (0, 4)
        maps = open("/proc/self/maps").read()
        assert "libw8a8_oracle" in maps
        assert "libw8a8_linear" not in maps, "the CUDA library was mapped by an oracle-side import"
        assert "paper_2606_14598_b200.binding" not in sys.modules
        pkg.status_string(0)                         # first touch of an entry point loads it
        assert "libw8a8_linear" in open("/proc/self/maps").read()
        print("independent")
    """) % ROOT
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and "independent" in r.stdout, r.stdout + r.stderr
