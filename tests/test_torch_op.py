"""The fused linear as a PyTorch custom operator: shape-only tracing without a GPU, and, on a GPU, a small MLP of
two such linears traced as ONE graph (no graph break at the quantized linears) and replayed from a CUDA graph,
checked against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2606_14598_b200 import inputs as synth


def test_operator_is_registered_and_traces_with_fake_tensors():
    from torch._subclasses.fake_tensor import FakeTensorMode

    from paper_2606_14598_b200 import torch_op
    assert hasattr(torch.ops.w8a8_b200, "linear_fused")
    with FakeTensorMode():
        A = torch.empty((3, 50, 64), dtype=torch.bfloat16)
        qw = torch.empty((24, 64), dtype=torch.int8)
        s_ch = torch.empty((24,), dtype=torch.float32)
        out = torch_op.linear_fused(A, qw, s_ch, None)          # the shape-only implementation: no kernel runs
        assert out.shape == (3, 50, 24) and out.dtype == torch.bfloat16
        with pytest.raises(Exception):
            torch_op.linear_fused(A.float(), qw, s_ch, None)


@pytest.mark.gpu
def test_compiled_mlp_has_no_graph_break_and_matches_the_oracle():
    import paper_2606_14598_b200 as w8
    from paper_2606_14598_b200.torch_op import W8A8Linear
    dev = "cuda:0"
    up, down = synth.LinearSpec("op_up", 300, 256, 512), synth.LinearSpec("op_down", 300, 512, 264)
    tu, td = synth.make_linear(up), synth.make_linear(down)

    class Mlp(torch.nn.Module):
        def __init__(self):
            super().__init__()
            self.up = W8A8Linear.from_float(tu["W"].to(dev), tu["bias"].to(dev))
            self.down = W8A8Linear.from_float(td["W"].to(dev), td["bias"].to(dev))

        def forward(self, x):
            return self.down(torch.relu(self.up(x)))        # an activation that is exact in bf16 (max with zero)

    mlp = Mlp()
    x = tu["A"].to(dev)
    eager = mlp(x)
    # the oracle's chain: linear, relu on the bf16 values, linear
    qwu, scu = oracle.quantize_weight_per_channel(tu["W"].numpy())
    qwd, scd = oracle.quantize_weight_per_channel(td["W"].numpy())
    h = oracle.linear_fused_bf16(synth.bf16_bits(tu["A"]), qwu, scu, tu["bias"].numpy())["out"]
    h_relu = np.where(h & 0x8000, 0, h).astype(np.uint16)
    ref = oracle.linear_fused_bf16(h_relu, qwd, scd, td["bias"].numpy())["out"]
    assert np.array_equal(synth.bf16_bits(eager.cpu()), ref)
    # one graph, no break at the quantized linears
    explanation = torch._dynamo.explain(mlp)(x)
    assert explanation.graph_break_count == 0 and explanation.graph_count == 1, str(explanation)
    compiled = torch.compile(mlp, fullgraph=True, backend="aot_eager")
    assert torch.equal(compiled(x), eager)
    # the calls allocate through torch only and enqueue on the current stream: replay from a CUDA graph
    static_x = x.clone()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        mlp(static_x)                                       # warm-up on the side stream
    torch.cuda.current_stream().wait_stream(s)
    with torch.cuda.graph(g):
        y = mlp(static_x)
    static_x.copy_(synth.make_activations(up, seed=3).to(dev))
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(y, mlp(static_x))
    assert w8.int8_sticky_status(clear=True) == 0
