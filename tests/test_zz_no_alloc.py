"""The allocation-free entry point, int8_linear_fused_static, against the workspace entry point and the oracle.

Some users of this library cannot allocate device memory when they call it (their own arena owns the GPU, or
an allocation's device-wide synchronisation is not acceptable where they call from). For them the library keeps
the scratch of the from-bf16 path in a fixed device array of its own; this file checks that the variant
computes the same bits as int8_linear_fused and as the CPU oracle, twice in a row (the array keeps the first
call's contents, which must not matter), also on a shape whose partial sums of the K-split land in the array,
that the call leaves the amount of free device memory unchanged, and that problems too large for the array
are refused.

The file name sorts last so that a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_14598_b200 as w8
from paper_2606_14598_b200 import binding
from paper_2606_14598_b200 import inputs as synth


def test_static_workspace_refuses_what_does_not_fit():
    # argument checks come before any CUDA call, so fake (aligned) addresses are never touched
    P = 0x10000
    lib = binding.raw()
    cap = binding.STATIC_WORKSPACE_BYTES
    assert w8.int8_linear_workspace_bytes(4608, 12288, 3072) <= cap < w8.int8_linear_workspace_bytes(4608, 3072, 12288)
    # M = 4608, K = 12288 needs ~57 MB of scratch: refused with the workspace error, nothing enqueued
    assert lib.int8_linear_fused_static(P, 12288, P, P, None, P, 3072, 4608, 3072, 12288, 0, None) == 4
    assert lib.int8_linear_fused_static(P, 64, P, P, None, P, 64, 0, 64, 64, 0, None) == 1       # M = 0


@pytest.mark.gpu
def test_static_workspace_matches_workspace_entry_point_twice_in_a_row():
    dev = "cuda:0"
    # three different problems, the largest first: each call finds the previous call's flags, scales, codes and
    # (third problem: deep K, its only tile is cut along K) partial sums and arrival counters still in the array
    specs = (synth.LinearSpec("static_a", 1000, 1024, 1544), synth.LinearSpec("static_b", 300, 384, 328, bias=False),
             synth.LinearSpec("static_c", 256, 8192, 264))
    for spec in specs:
        t = synth.make_linear(spec)
        A = t["A"].to(dev)
        bias = None if t["bias"] is None else t["bias"].to(dev)
        qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(t["W"].numpy())
        ref = oracle.linear_fused_bf16(synth.bf16_bits(t["A"]), qw_ref, s_ch_ref, None if t["bias"] is None else t["bias"].numpy())
        qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(dev))
        ws = w8.alloc_workspace(spec.M, spec.N, spec.K, w8.ACT_BF16, dev)
        want = w8.int8_linear_fused(A, qw, s_ch, bias, workspace=ws)
        assert w8.int8_check_status(ws) == 0
        if spec.name == "static_c":                        # the static entry hands the planner the whole array
            plan = w8.int8_linear_plan(spec.M, spec.N, spec.K, w8.ACT_BF16, binding.STATIC_WORKSPACE_BYTES)
            assert plan["split_parts"] >= 2, plan
        out = torch.empty_like(want)                       # the caller's own output buffer
        for call in range(2):                              # two calls in a row through the C ABI
            out.fill_(7.0)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            w8.int8_linear_fused_static(A, qw, s_ch, bias, out=out, sync_and_check=True)
            if call == 1:                                  # (the very first call on a device loads the array's module)
                assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the free device memory"
            got, same = synth.bf16_bits(out.cpu()), synth.bf16_bits(want.cpu())
            d = np.abs(np.where(got & 0x8000, -(got & 0x7FFF).astype(np.int32), got.astype(np.int32)) -
                       np.where(ref["out"] & 0x8000, -(ref["out"] & 0x7FFF).astype(np.int32), ref["out"].astype(np.int32)))
            assert d.max() <= 1                            # the tolerance of the parity tests: 1 bf16 ulp of the oracle
            assert np.array_equal(got, ref["out"])         # same operation order as the oracle: in fact the same bits
            assert np.array_equal(got, same)               # and the same bits as the workspace entry point
    # the asynchronous form (no synchronize inside the call)
    out2 = w8.int8_linear_fused_static(A, qw, s_ch, bias)
    torch.cuda.synchronize()
    assert torch.equal(out2, want)
