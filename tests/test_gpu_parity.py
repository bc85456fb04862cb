"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

Bars: int8 codes, fp32 scales and int32 accumulators bit-exact; bf16 outputs within 1 bf16 ulp
(ordered-integer distance of the bit patterns, +0 == -0) with cosine >= 0.99999. Because the
kernels follow the oracle's operation order, the bf16 outputs are in fact expected to be equal
bit for bit, and the tests assert that too.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_14598_b200 as w8
from paper_2606_14598_b200 import inputs as synth

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def n_tc_configs():
    return w8.num_configs() - 1          # the last configuration is the CUDA-core path


@pytest.fixture(autouse=True)
def _reset_config():
    w8.force_config(-1)
    yield
    w8.force_config(-1)


def ordered(bits):
    b = bits.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b)


def bits_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def assert_bf16_close(got_bits, ref_bits, exact=True):
    assert got_bits.shape == ref_bits.shape
    d = np.abs(ordered(got_bits) - ordered(ref_bits))
    assert d.max() <= 1, f"max ulp distance {d.max()} at {np.unravel_index(d.argmax(), d.shape)}"
    g, r = bits_f64(got_bits).ravel(), bits_f64(ref_bits).ravel()
    assert np.isfinite(g).all()
    nz = r != 0
    if nz.any():
        rel = np.abs(g[nz] - r[nz]) / np.abs(r[nz])
        assert rel.max() <= 2.0 ** -7
    den = np.sqrt((g * g).sum() * (r * r).sum())
    if den > 0:
        assert (g * r).sum() / den >= 0.99999
    if exact:
        assert (d == 0).all(), f"{int((d != 0).sum())} of {d.size} outputs differ by one ulp"


def check_status(ws):
    st = w8.int8_check_status(ws)
    assert st == 0, w8.status_string(st)


def rand_codes(rng, shape, lo=-127):
    return rng.integers(lo, 128, shape, dtype=np.int8)


# ------------------------------------------------------------------------------- quantizers (T1)

@pytest.mark.parametrize("M,K", [(1, 16), (7, 48), (33, 2048), (300, 3072), (9, 4096), (5, 8192), (40, 12288),
                                 (3, 16384), (3, 16400), (2, 40000), (150, 53248), (3, 57600), (3, 57616),
                                 (2, 66000), (2, 133136)])
def test_act_quantizer_bit_exact(M, K):
    spec = synth.LinearSpec(f"q{M}x{K}", M, K, 8, outlier_frac=0.01 if K >= 256 else 0.0)
    A = synth.make_activations(spec)
    if M > 2:
        A[1] = 0                                   # an all-zero token
    qa_ref, s_ref = oracle.quantize_act_per_token(synth.bf16_bits(A))
    qa, s = w8.int8_quantize_act_per_token(A.to(DEV))
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(qa.cpu().numpy(), qa_ref)


def test_act_quantizer_every_bf16_value_against_many_scales():
    """Exhaustive in x: every finite bf16 value not above the row's absmax, for 320 different absmax
    values (random ones, all-ones and all-zeros mantissas, tiny and huge exponents). bf16 inputs make
    exact rounding ties common, so this is where a quotient that is off by one ulp would show."""
    rng = np.random.default_rng(2024)
    pats = np.arange(65536, dtype=np.uint32)
    finite = (pats & 0x7F80) != 0x7F80
    vals = np.where(finite, pats, 0).astype(np.uint16)                      # NaN / Inf patterns -> +0
    mags = (vals & 0x7FFF).astype(np.int64)
    amax_bits = np.concatenate([
        rng.integers(0x3000, 0x4F00, 256),                                   # ordinary magnitudes
        np.array([0x3F80, 0x3FFF, 0x407F, 0x42FE, 0x4000, 0x3F7F, 0x437F, 0x3E00]),   # 1, all-ones mantissas, 127, 255 ...
        rng.integers(0x0080, 0x0800, 24), rng.integers(0x7000, 0x7F7F, 32)]).astype(np.int64)   # tiny / huge
    rows = []
    for ab in amax_bits:
        row = np.where(mags <= ab, vals, 0).astype(np.uint16)
        row = row.reshape(8, 8192).copy()
        row[:, 0] = ab                                                       # every row carries its absmax
        rows.append(row)
    A_bits = np.ascontiguousarray(np.concatenate(rows, axis=0))
    qa_ref, s_ref = oracle.quantize_act_per_token(A_bits)
    A = synth.bits_to_bf16(A_bits).to(DEV)
    qa, s = w8.int8_quantize_act_per_token(A)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    got = qa.cpu().numpy()
    bad = np.argwhere(got != qa_ref)
    assert bad.size == 0, f"{len(bad)} codes differ, first at {bad[0]}: got {got[tuple(bad[0])]} want {qa_ref[tuple(bad[0])]}"


def test_act_quantizer_gelu_rows_and_row_stride():
    spec = synth.LinearSpec("qg", 70, 1024, 8, act="gelu", outlier_frac=0.0)
    A = synth.make_activations(spec)
    qa_ref, s_ref = oracle.quantize_act_per_token(synth.bf16_bits(A))
    wide = torch.full((70, 1024 + 64), 7.0, dtype=torch.bfloat16, device=DEV)
    wide[:, :1024] = A.to(DEV)
    qa, s = w8.int8_quantize_act_per_token(wide[:, :1024])           # lda = 1088
    assert np.array_equal(s.cpu().numpy(), s_ref) and np.array_equal(qa.cpu().numpy(), qa_ref)


def test_act_quantizer_hand_ties_on_device():
    x = torch.tensor([[127, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 63.5, 126.5, -126.5, 0.375, 0.625, -127, 3, 0, 0]],
                     dtype=torch.bfloat16)
    qa, s = w8.int8_quantize_act_per_token(x.to(DEV))
    assert s.item() == 1.0
    assert qa.cpu().tolist() == [[127, 0, 2, 2, 0, -2, -2, 64, 126, -126, 0, 1, -127, 3, 0, 0]]


@pytest.mark.parametrize("N,K", [(5, 16), (256, 256), (100, 3072), (17, 12288), (3, 16400)])
def test_weight_quantizer_bit_exact(N, K):
    spec = synth.LinearSpec(f"w{N}x{K}", 8, K, N)
    W = synth.make_weight(spec)
    if N > 2:
        W[2] = 0
    qw_ref, s_ref = oracle.quantize_weight_per_channel(W.numpy())
    qw, s = w8.int8_quantize_weight_per_channel(W.to(DEV))
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(qw.cpu().numpy(), qw_ref)


# ------------------------------------------------------------------------------- SmoothQuant hook

def smooth_factor(K, seed):
    rng = np.random.default_rng(seed)
    return (rng.random(K) * 3 + 0.1).astype(np.float32)


@pytest.mark.parametrize("M,K", [(1, 16), (33, 2048), (300, 3072), (40, 12288), (3, 40000), (150, 53248), (2, 66000)])
def test_act_quantizer_smooth_bit_exact(M, K):
    spec = synth.LinearSpec(f"qs{M}x{K}", M, K, 8, outlier_frac=0.01 if K >= 256 else 0.0)
    A = synth.make_activations(spec)
    mult = smooth_factor(K, K)
    qa_ref, s_ref = oracle.quantize_act_per_token_smooth(synth.bf16_bits(A), mult)
    qa, s = w8.int8_quantize_act_per_token_smooth(A.to(DEV), torch.from_numpy(mult).to(DEV))
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(qa.cpu().numpy(), qa_ref)


@pytest.mark.parametrize("N,K", [(100, 3072), (17, 12288), (3, 16400)])
def test_weight_quantizer_smooth_bit_exact(N, K):
    W = synth.make_weight(synth.LinearSpec(f"ws{N}x{K}", 8, K, N))
    mult = smooth_factor(K, N)
    qw_ref, s_ref = oracle.quantize_weight_per_channel_smooth(W.numpy(), mult)
    qw, s = w8.int8_quantize_weight_per_channel_smooth(W.to(DEV), torch.from_numpy(mult).to(DEV))
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(qw.cpu().numpy(), qw_ref)


def test_fused_smooth_matches_oracle():
    spec = synth.LinearSpec("fsmooth", 1000, 1024, 1544, outlier_frac=0.02)
    t = synth.make_linear(spec)
    A_bits = synth.bf16_bits(t["A"])
    W, b = t["W"].numpy(), t["bias"].numpy()
    # alpha = 0.5 factors from the tensors themselves (calibration stands outside the path)
    ax = np.abs(t["A"].float().numpy()).max(axis=0).astype(np.float64)
    aw = np.abs(W).max(axis=0).astype(np.float64)
    sm = np.sqrt(ax / aw)
    a_mult, w_mult = (1.0 / sm).astype(np.float32), sm.astype(np.float32)
    qw_ref, s_ch_ref = oracle.quantize_weight_per_channel_smooth(W, w_mult)
    ref = oracle.linear_fused_bf16_smooth(A_bits, a_mult, qw_ref, s_ch_ref, b)
    qw, s_ch = w8.int8_quantize_weight_per_channel_smooth(t["W"].to(DEV), torch.from_numpy(w_mult).to(DEV))
    assert np.array_equal(qw.cpu().numpy(), qw_ref) and np.array_equal(s_ch.cpu().numpy(), s_ch_ref)
    ws = w8.alloc_workspace(spec.M, spec.N, spec.K, w8.ACT_BF16, DEV)
    out = w8.int8_linear_fused_smooth(t["A"].to(DEV), torch.from_numpy(a_mult).to(DEV), qw, s_ch, t["bias"].to(DEV),
                                      workspace=ws)
    check_status(ws)
    s_off, q_off = w8.int8_linear_workspace_offsets(spec.M, spec.K)
    qa = ws[q_off:q_off + spec.M * spec.K].view(torch.int8).view(spec.M, spec.K).cpu().numpy()
    assert np.array_equal(qa, ref["qa"])
    assert_bf16_close(synth.bf16_bits(out.cpu()), ref["out"])


# ------------------------------------------------------------------------------- raw accumulators (T2)

ACC_SHAPES = [
    (128, 256, 128),     # exactly one tile, one k-block
    (128, 256, 16), (128, 256, 32), (128, 256, 48), (128, 256, 144), (128, 128, 400),
    (1, 8, 16), (17, 8, 64), (129, 264, 160),
    (300, 328, 384),     # ragged in M and N, several tiles
    (640, 10240, 256),   # 200 tiles of 128x256: more than one tile per CTA, both accumulator buffers
    (2816, 3072, 512),
]


@pytest.mark.parametrize("M,N,K", ACC_SHAPES)
def test_accumulators_bit_exact_all_tensor_core_configs(M, N, K):
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    qa, qw = rand_codes(rng, (M, K)), rand_codes(rng, (N, K))
    ref = oracle.gemm_i32(qa, qw)
    dqa, dqw = torch.from_numpy(qa).to(DEV), torch.from_numpy(qw).to(DEV)
    for cfg in range(w8.num_configs()):
        if cfg == n_tc_configs() and M * N * K > 2 ** 31:
            continue                                    # the CUDA-core path is slow on big shapes
        w8.force_config(cfg)
        ws = w8.alloc_workspace(M, N, K, w8.ACT_INT8, DEV)
        acc = w8.int8_gemm_i32_debug(dqa, dqw, ws)
        check_status(ws)
        assert np.array_equal(acc.cpu().numpy(), ref), f"config {cfg}: {w8.config_name(cfg)}"


def test_accumulators_overflow_edge_and_minus_128():
    # K * 127^2 just below 2^31, every product at its extreme
    K = 133136
    qa = np.full((130, K), 127, np.int8)
    qa[1::2] = -127
    qw = np.full((16, K), 127, np.int8)
    qw[3] = -127
    dqa, dqw = torch.from_numpy(qa).to(DEV), torch.from_numpy(qw).to(DEV)
    want = (qa[:, :1].astype(np.int64) * qw[:, :1].astype(np.int64).T) * K
    assert abs(want).max() == K * 16129 < 2 ** 31
    for cfg in range(n_tc_configs()):
        w8.force_config(cfg)
        acc = w8.int8_gemm_i32_debug(dqa, dqw)
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), want), cfg
    # -128 codes are tolerated and exact while K <= 131071
    w8.force_config(-1)
    rng = np.random.default_rng(3)
    qa2, qw2 = rand_codes(rng, (200, 512), lo=-128), rand_codes(rng, (264, 512), lo=-128)
    qa2[0, :] = -128
    qw2[0, :] = -128
    acc = w8.int8_gemm_i32_debug(torch.from_numpy(qa2).to(DEV), torch.from_numpy(qw2).to(DEV))
    assert np.array_equal(acc.cpu().numpy(), oracle.gemm_i32(qa2, qw2))
    assert acc[0, 0].item() == 512 * 16384


def test_accumulators_match_library_int_mm():
    # the paper's own gate: the integer accumulation equals an independent integer matmul
    rng = np.random.default_rng(8)
    qa = torch.from_numpy(rand_codes(rng, (2816, 3072))).to(DEV)
    qw = torch.from_numpy(rand_codes(rng, (3072, 3072))).to(DEV)
    want = torch._int_mm(qa, qw.t())
    for cfg in range(n_tc_configs()):
        w8.force_config(cfg)
        assert torch.equal(w8.int8_gemm_i32_debug(qa, qw), want), cfg


# ------------------------------------------------------------------------------- fused output (T3)

FUSED_SHAPES = [(128, 256, 256), (300, 384, 328), (129, 3072, 264), (1000, 1024, 1536), (640, 256, 10240)]


@pytest.mark.parametrize("M,K,N", FUSED_SHAPES)
@pytest.mark.parametrize("use_bias", [True, False])
def test_fused_from_bf16_matches_oracle(M, K, N, use_bias):
    spec = synth.LinearSpec(f"f{M}x{K}x{N}", M, K, N, bias=use_bias)
    t = synth.make_linear(spec)
    if M > 4:
        t["A"][3] = 0                                   # zero token: output row equals the bias
    qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(t["W"].numpy())
    bias_np = t["bias"].numpy() if use_bias else None
    ref = oracle.linear_fused_bf16(synth.bf16_bits(t["A"]), qw_ref, s_ch_ref, bias_np)
    qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
    assert np.array_equal(qw.cpu().numpy(), qw_ref) and np.array_equal(s_ch.cpu().numpy(), s_ch_ref)
    bias = t["bias"].to(DEV) if use_bias else None
    A = t["A"].to(DEV)
    for cfg in range(w8.num_configs()):
        w8.force_config(cfg)
        ws = w8.alloc_workspace(M, N, K, w8.ACT_BF16, DEV)
        out = w8.int8_linear_fused(A, qw, s_ch, bias, workspace=ws)
        check_status(ws)
        # the intermediate tensors the call leaves in the workspace
        s_off, q_off = w8.int8_linear_workspace_offsets(M, K)
        s_tok = ws[s_off:s_off + 4 * M].view(torch.float32).cpu().numpy()
        qa = ws[q_off:q_off + M * K].view(torch.int8).view(M, K).cpu().numpy()
        assert np.array_equal(s_tok, ref["s_tok"]) and np.array_equal(qa, ref["qa"]), cfg
        assert_bf16_close(synth.bf16_bits(out.cpu()), ref["out"])
    if M > 4 and use_bias:
        zero_row = synth.bf16_bits(out.cpu())[3]
        assert np.array_equal(zero_row, synth.bf16_bits(t["bias"].to(torch.bfloat16)))


def test_fused_from_int8_with_row_stride_and_guard_bands():
    M, K, N = 200, 512, 328
    rng = np.random.default_rng(21)
    qa, qw = rand_codes(rng, (M, K)), rand_codes(rng, (N, K))
    s_tok = (rng.random(M) * 0.05 + 0.01).astype(np.float32)
    s_ch = (rng.random(N) * 0.0008 + 0.0002).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.01).astype(np.float32)
    ref = oracle.linear_fused_int8(qa, s_tok, qw, s_ch, bias)
    qa_wide = torch.zeros((M, K + 64), dtype=torch.int8, device=DEV)
    qa_wide[:, :K] = torch.from_numpy(qa).to(DEV)
    SENT = -2.0
    canvas = torch.full((M + 40, N + 56), SENT, dtype=torch.bfloat16, device=DEV)   # output lives inside a larger buffer
    for cfg in range(w8.num_configs()):
        w8.force_config(cfg)
        canvas.fill_(SENT)
        out_view = canvas[8:8 + M, 16:16 + N]
        ws = w8.alloc_workspace(M, N, K, w8.ACT_INT8, DEV)
        w8.int8_linear_fused(qa_wide[:, :K], torch.from_numpy(qw).to(DEV), torch.from_numpy(s_ch).to(DEV),
                             torch.from_numpy(bias).to(DEV), s_tok=torch.from_numpy(s_tok).to(DEV), out=out_view,
                             workspace=ws)
        check_status(ws)
        assert_bf16_close(synth.bf16_bits(out_view.contiguous().cpu()), ref["out"])
        mask = torch.ones_like(canvas, dtype=torch.bool)
        mask[8:8 + M, 16:16 + N] = False
        assert (canvas[mask] == SENT).all(), f"config {cfg} wrote outside its output"


def test_fused_from_bf16_with_row_stride_no_bias_and_k_split():
    # activations that are a column slice of a wider tensor (row stride > K), no bias, on a shape that is cut along K
    spec = synth.LinearSpec("strided", 260, 8192, 520, bias=False)
    t = synth.make_linear(spec)
    qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(t["W"].numpy())
    ref = oracle.linear_fused_bf16(synth.bf16_bits(t["A"]), qw_ref, s_ch_ref, None)
    qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
    wide = torch.full((spec.M, spec.K + 72), 7.0, dtype=torch.bfloat16, device=DEV)
    wide[:, 8:8 + spec.K] = t["A"].to(DEV)
    A_view = wide[:, 8:8 + spec.K]
    assert A_view.stride(0) == spec.K + 72 and A_view.data_ptr() % 16 == 0
    ws = w8.alloc_workspace(spec.M, spec.N, spec.K, w8.ACT_BF16, DEV)
    assert w8.int8_linear_plan(spec.M, spec.N, spec.K, w8.ACT_BF16, ws.numel())["split_parts"] >= 2
    out = w8.int8_linear_fused(A_view, qw, s_ch, None, workspace=ws)
    check_status(ws)
    assert_bf16_close(synth.bf16_bits(out.cpu()), ref["out"])
    assert (wide[:, :8] == 7.0).all() and (wide[:, 8 + spec.K:] == 7.0).all()


@pytest.mark.parametrize("M,K,N", [(1, 3072, 2048), (2, 3072, 2048), (5, 3072, 2048), (16, 3072, 2048),
                                   (3, 3072, 2056), (4, 1024, 4104), (2, 6144, 1032), (2, 16, 1024), (2, 12288, 1544),
                                   (2, 3072, 18432)])
def test_skinny_m_path(M, K, N):
    # M <= 4 with enough weight rows: the weight-streaming kernel (ring of bulk copies); M = 5 and rows too long for a
    # three-stage ring: the register kernel; M = 16: the tensor-core path
    spec = synth.LinearSpec(f"skinny{M}x{K}x{N}", M, K, N, outlier_frac=0.0)
    t = synth.make_linear(spec)
    qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(t["W"].numpy())
    ref = oracle.linear_fused_bf16(synth.bf16_bits(t["A"]), qw_ref, s_ch_ref, t["bias"].numpy())
    qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
    ws = w8.alloc_workspace(M, spec.N, spec.K, w8.ACT_BF16, DEV)
    out, rowmax = w8.int8_linear_fused_rowmax(t["A"].to(DEV), qw, s_ch, t["bias"].to(DEV), workspace=ws)
    check_status(ws)
    assert_bf16_close(synth.bf16_bits(out.cpu()), ref["out"])
    assert np.array_equal(rowmax.cpu().numpy(), oracle.row_absmax_bf16(ref["out"]))
    s_off, q_off = w8.int8_linear_workspace_offsets(M, K)
    qa = ws[q_off:q_off + M * K].view(torch.int8).view(M, K)
    acc = w8.int8_gemm_i32_debug(qa, qw)
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])


def test_run_to_run_identical_and_host_buffer_entry_point():
    spec = synth.LinearSpec("rr", 1100, 1024, 1544)
    t = synth.make_linear(spec)
    qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
    A, bias = t["A"].to(DEV), t["bias"].to(DEV)
    ws = w8.alloc_workspace(spec.M, spec.N, spec.K, w8.ACT_BF16, DEV)
    first = w8.int8_linear_fused(A, qw, s_ch, bias, workspace=ws).clone()
    for _ in range(5):
        assert torch.equal(w8.int8_linear_fused(A, qw, s_ch, bias, workspace=ws), first)
    check_status(ws)
    A_host = t["A"].pin_memory()
    out_host = torch.empty((spec.M, spec.N), dtype=torch.bfloat16).pin_memory()
    d_A, d_out = torch.empty_like(A), torch.empty_like(first)
    w8.int8_linear_fused_host(A_host, d_A, qw, s_ch, bias, d_out, out_host, ws)
    check_status(ws)
    assert torch.equal(out_host, first.cpu())


# ------------------------------------------------------------------------------- stored digests

def test_cuda_results_match_stored_oracle_digests():
    # tests/golden/oracle_hashes.json holds SHA-256 digests of what the CPU oracle computed from the seeded inputs
    # (written by tests/golden/make_oracle_hashes.py, which never touches the CUDA library): the device must
    # produce the same bytes, whatever machine the digests were written on
    import hashlib
    import importlib.util
    import json
    import os
    here = os.path.dirname(os.path.abspath(__file__))
    mspec = importlib.util.spec_from_file_location("make_oracle_hashes", os.path.join(here, "golden", "make_oracle_hashes.py"))
    mod = importlib.util.module_from_spec(mspec)
    mspec.loader.exec_module(mod)
    stored = json.load(open(os.path.join(here, "golden", "oracle_hashes.json")))

    def digest(t):
        return hashlib.sha256(np.ascontiguousarray(t.cpu().numpy()).tobytes()).hexdigest()

    for spec in mod.CASES:
        want = stored[spec.name]
        t = synth.make_linear(spec)
        assert mod.digest(synth.bf16_bits(t["A"])) == want["A"], "the generator's stream differs on this machine"
        qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
        bias = None if t["bias"] is None else t["bias"].to(DEV)
        ws = w8.alloc_workspace(spec.M, spec.N, spec.K, w8.ACT_BF16, DEV)
        out = w8.int8_linear_fused(t["A"].to(DEV), qw, s_ch, bias, workspace=ws)
        check_status(ws)
        s_off, q_off = w8.int8_linear_workspace_offsets(spec.M, spec.K)
        s_tok = ws[s_off:s_off + 4 * spec.M].view(torch.float32)
        qa = ws[q_off:q_off + spec.M * spec.K].view(torch.int8).view(spec.M, spec.K)
        acc = w8.int8_gemm_i32_debug(qa, qw)
        got = {"qw": digest(qw), "s_ch": digest(s_ch), "qa": digest(qa), "s_tok": digest(s_tok), "acc": digest(acc),
               "out": digest(out.view(torch.int16))}
        for key, val in got.items():
            assert val == want[key], f"{spec.name}: {key}"


# ------------------------------------------------------------------------------- K-split of the partial wave

# (M, N, K, configuration): shapes whose last (or only) wave of tiles leaves SMs idle, so that its tiles
# are cut along K and the int32 partial sums are added up by the part that finishes last
SPLIT_SHAPES = [
    (256, 512, 2048, 2),      # two pair tiles, two parts each
    (300, 520, 2064, 2),      # ragged M, N and K
    (256, 256, 8192, 2),      # one tile in eight parts
    (130, 264, 4096, 0),      # one CTA per tile
    (300, 400, 4096, 4),      # 192-column tiles
    (512, 5120, 2048, 3),     # 80 pair tiles on 74 pairs: a whole wave, then 6 tiles in parts
    (512, 4864, 2048, 1),     # 152 tiles on 148 CTAs
]


@pytest.mark.parametrize("M,N,K,cfg", SPLIT_SHAPES)
def test_k_split_accumulators_and_outputs_bit_exact(M, N, K, cfg):
    rng = np.random.default_rng(M + 3 * N + 5 * K + cfg)
    qa, qw = rand_codes(rng, (M, K)), rand_codes(rng, (N, K))
    s_tok = (rng.random(M) * 0.05 + 0.01).astype(np.float32)
    s_ch = (rng.random(N) * 0.0008 + 0.0002).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.01).astype(np.float32)
    ref = oracle.linear_fused_int8(qa, s_tok, qw, s_ch, bias)
    dev = [torch.from_numpy(a).to(DEV) for a in (qa, qw, s_tok, s_ch, bias)]
    ws = w8.alloc_workspace(M, N, K, w8.ACT_INT8, DEV)
    ws_big = torch.empty(ws.numel() + (32 << 20), dtype=torch.uint8, device=DEV)   # room for any split
    for forced, want_split in ((cfg, True), (cfg + 0x100, False)):
        w8.force_config(forced)
        plan = w8.int8_linear_plan(M, N, K, w8.ACT_INT8, ws_big.numel())
        assert plan["config"] == cfg and (plan["split_parts"] >= 2) == want_split, plan
        ws_big.fill_(0x5A)                              # the scratch needs no initialisation
        acc = w8.int8_gemm_i32_debug(dev[0], dev[1], ws_big)
        check_status(ws_big)
        assert np.array_equal(acc.cpu().numpy(), ref["acc"]), plan
        for _ in range(2):                              # twice on the same scratch
            out = w8.int8_linear_fused(dev[0], dev[1], dev[3], dev[4], s_tok=dev[2], workspace=ws_big)
            check_status(ws_big)
            assert_bf16_close(synth.bf16_bits(out.cpu()), ref["out"])
    # a workspace of the minimum size turns the split off and gives the same output
    w8.force_config(cfg)
    ws_min = torch.empty(w8.int8_linear_workspace_min_bytes(M, N, K, w8.ACT_INT8), dtype=torch.uint8, device=DEV)
    assert w8.int8_linear_plan(M, N, K, w8.ACT_INT8, ws_min.numel())["split_parts"] == 0
    out = w8.int8_linear_fused(dev[0], dev[1], dev[3], dev[4], s_tok=dev[2], workspace=ws_min)
    check_status(ws_min)
    assert_bf16_close(synth.bf16_bits(out.cpu()), ref["out"])


def test_k_split_from_bf16_automatic_choice():
    # few tiles and a deep K: the automatic choice cuts along K (when the workspace has the room it asks for)
    spec = synth.LinearSpec("split_bf16", 500, 8192, 776)
    t = synth.make_linear(spec)
    qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(t["W"].numpy())
    ref = oracle.linear_fused_bf16(synth.bf16_bits(t["A"]), qw_ref, s_ch_ref, t["bias"].numpy())
    qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
    ws = w8.alloc_workspace(spec.M, spec.N, spec.K, w8.ACT_BF16, DEV)
    assert ws.numel() > w8.int8_linear_workspace_min_bytes(spec.M, spec.N, spec.K, w8.ACT_BF16)
    assert w8.int8_linear_plan(spec.M, spec.N, spec.K, w8.ACT_BF16, ws.numel())["split_parts"] >= 2
    out = w8.int8_linear_fused(t["A"].to(DEV), qw, s_ch, t["bias"].to(DEV), workspace=ws)
    check_status(ws)
    assert_bf16_close(synth.bf16_bits(out.cpu()), ref["out"])
    w8.force_config(-2)                                 # same shape, never cut
    assert w8.int8_linear_plan(spec.M, spec.N, spec.K, w8.ACT_BF16, ws.numel())["split_parts"] == 0
    out2 = w8.int8_linear_fused(t["A"].to(DEV), qw, s_ch, t["bias"].to(DEV), workspace=ws)
    check_status(ws)
    assert torch.equal(out, out2)


# ------------------------------------------------------------------------------- quantizer fused into its producer

# Shapes that between them reach every way the staged quantizer runs its ring: a barrier pair per row slot fed by
# 16 / 4 / 2 / 1 producer lanes or a pair per stage, one or two CTAs per SM (two from 8 row groups per SM on), a last
# group with fewer rows than a stage has slots.
@pytest.mark.parametrize("M,K", [(19003, 1024), (37889, 512), (10007, 2048), (9497, 1536), (9481, 3072), (4737, 4096),
                                 (4740, 6144), (2369, 12288), (1185, 16384), (9473, 16)])
def test_act_quantizer_every_ring_variant_against_oracle(M, K):
    rng = np.random.default_rng(M + K)
    scale = rng.choice(np.array([0.01, 1.0, 50.0], dtype=np.float32), size=(M, 1))
    A = torch.from_numpy(rng.standard_normal((M, K), dtype=np.float32) * scale).to(torch.bfloat16)
    A[int(rng.integers(0, M))] = 0
    bits = synth.bf16_bits(A)
    qa_ref, s_ref = oracle.quantize_act_per_token(bits)
    dA = A.to(DEV)
    qa, s = w8.int8_quantize_act_per_token(dA)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(qa.cpu().numpy(), qa_ref)
    qa1, s1 = w8.int8_quantize_act_per_token_given_absmax(dA, torch.from_numpy(oracle.row_absmax_bf16(bits)).to(DEV))
    assert np.array_equal(s1.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(qa1.cpu().numpy(), qa_ref)
    assert w8.int8_sticky_status(clear=True) == 0


@pytest.mark.parametrize("M,K", [(1, 16), (33, 2048), (300, 3072), (40, 12288), (3, 40000), (6, 53248), (2, 66000)])
def test_one_pass_quantizer_with_the_absmax_handed_in(M, K):
    spec = synth.LinearSpec(f"q1p{M}x{K}", M, K, 8, outlier_frac=0.01 if K >= 256 else 0.0)
    A = synth.make_activations(spec)
    if M > 2:
        A[1] = 0
    bits = synth.bf16_bits(A)
    rowmax = oracle.row_absmax_bf16(bits)
    qa_ref, s_ref = oracle.quantize_act_per_token(bits)
    # the row's own absmax: the one-pass quantizer equals the two-pass one (oracle and device)
    qa, s = w8.int8_quantize_act_per_token_given_absmax(A.to(DEV), torch.from_numpy(rowmax).to(DEV))
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(qa.cpu().numpy(), qa_ref)
    # a larger absmax (allowed): against the oracle's given-absmax function
    bigger = (rowmax * np.float32(1.75) + np.float32(0.125)).astype(np.float32)
    qa_ref2, s_ref2 = oracle.quantize_act_per_token_given_absmax(bits, bigger)
    qa2, s2 = w8.int8_quantize_act_per_token_given_absmax(A.to(DEV), torch.from_numpy(bigger).to(DEV))
    assert np.array_equal(s2.cpu().numpy().view(np.uint32), s_ref2.view(np.uint32))
    assert np.array_equal(qa2.cpu().numpy(), qa_ref2)


@pytest.mark.parametrize("cfg", [-1, 0, 2, 5, "simt"])
def test_row_maxima_from_the_epilogue_feed_the_next_linears_quantizer(cfg):
    """Two chained linears: the first also reports the largest magnitude it wrote per token, the second quantizes
    that output in one pass with it. Every tensor against the oracle: the maxima equal the row absmax of the
    first output, and the chain equals the two-pass path bit for bit."""
    M, K1, N1, N2 = 300, 1024, 1552, 520
    l1, l2 = synth.LinearSpec("chain1", M, K1, N1), synth.LinearSpec("chain2", M, N1, N2, bias=False)
    t1, W2 = synth.make_linear(l1), synth.make_weight(l2)
    t1["A"][5] = 0                                      # a zero token: its output row is the bias
    qw1_ref, sch1_ref = oracle.quantize_weight_per_channel(t1["W"].numpy())
    qw2_ref, sch2_ref = oracle.quantize_weight_per_channel(W2.numpy())
    r1 = oracle.linear_fused_bf16(synth.bf16_bits(t1["A"]), qw1_ref, sch1_ref, t1["bias"].numpy())
    rowmax_ref = oracle.row_absmax_bf16(r1["out"])
    qa2_ref, stok2_ref = oracle.quantize_act_per_token_given_absmax(r1["out"], rowmax_ref)
    r2 = oracle.linear_fused_int8(qa2_ref, stok2_ref, qw2_ref, sch2_ref, None)
    assert np.array_equal(r2["out"], oracle.linear_fused_bf16(r1["out"], qw2_ref, sch2_ref, None)["out"])

    qw1, sch1 = w8.int8_quantize_weight_per_channel(t1["W"].to(DEV))
    qw2, sch2 = w8.int8_quantize_weight_per_channel(W2.to(DEV))
    w8.force_config(n_tc_configs() if cfg == "simt" else cfg)
    ws1 = w8.alloc_workspace(M, N1, K1, w8.ACT_BF16, DEV)
    ws2 = w8.alloc_workspace(M, N2, N1, w8.ACT_BF16, DEV)
    y1, rowmax = w8.int8_linear_fused_rowmax(t1["A"].to(DEV), qw1, sch1, t1["bias"].to(DEV), workspace=ws1)
    y2, rowmax2 = w8.int8_linear_fused_rowmax(y1, qw2, sch2, None, workspace=ws2, rowmax_in=rowmax)
    check_status(ws1)
    check_status(ws2)
    assert np.array_equal(synth.bf16_bits(y1.cpu()), r1["out"])
    assert np.array_equal(rowmax.cpu().numpy().view(np.uint32), rowmax_ref.view(np.uint32))
    s_off, q_off = w8.int8_linear_workspace_offsets(M, N1)
    assert np.array_equal(ws2[q_off:q_off + M * N1].view(torch.int8).view(M, N1).cpu().numpy(), qa2_ref)
    assert np.array_equal(ws2[s_off:s_off + 4 * M].view(torch.float32).cpu().numpy(), stok2_ref)
    assert_bf16_close(synth.bf16_bits(y2.cpu()), r2["out"])
    assert np.array_equal(rowmax2.cpu().numpy(), oracle.row_absmax_bf16(r2["out"]))
    # input and output maxima must not share memory
    lib = w8.binding.raw()
    rc = lib.int8_linear_fused_given_absmax(y1.data_ptr(), N1, rowmax.data_ptr(), qw2.data_ptr(), sch2.data_ptr(), None,
                                            y2.data_ptr(), N2, rowmax.data_ptr(), M, N2, N1, ws2.data_ptr(), ws2.numel(), None)
    assert rc == 1


def test_row_maxima_from_a_k_split_tile():
    # the part that finishes a tile cut along K runs the epilogue from the summed slab: the maxima come from there too
    spec = synth.LinearSpec("rowmax_split", 256, 8192, 264)
    t = synth.make_linear(spec)
    qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(t["W"].numpy())
    ref = oracle.linear_fused_bf16(synth.bf16_bits(t["A"]), qw_ref, s_ch_ref, t["bias"].numpy())
    qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
    ws = w8.alloc_workspace(spec.M, spec.N, spec.K, w8.ACT_BF16, DEV)
    assert w8.int8_linear_plan(spec.M, spec.N, spec.K, w8.ACT_BF16, ws.numel())["split_parts"] >= 2
    y, rowmax = w8.int8_linear_fused_rowmax(t["A"].to(DEV), qw, s_ch, t["bias"].to(DEV), workspace=ws)
    check_status(ws)
    assert np.array_equal(synth.bf16_bits(y.cpu()), ref["out"])
    assert np.array_equal(rowmax.cpu().numpy(), oracle.row_absmax_bf16(ref["out"]))


# ------------------------------------------------------------------------------- wide items (two sub-tiles sharing A)

WIDE_SHAPES = [
    # (M, N, K, wide items per row block; None = the planner's choice)
    (600, 1536, 512, None), (600, 1536, 512, 0), (600, 1536, 512, 1), (600, 1536, 512, 2), (600, 1536, 512, 3),
    (300, 1288, 400, 2),      # ragged N: the last column block is partly outside, K tail inside a stage
    (300, 1288, 400, 3),      # ... and inside the second half of a wide item
    (130, 264, 160, 1),       # one wide item whose second half lies almost entirely outside N
    (2816, 3072, 1024, 4),    # 11 row blocks x (4 wide + 4 narrow): every group gets several items of both kinds
    (4608, 3072, 256, 6),     # all wide, 108 items on 74 groups
]


@pytest.mark.parametrize("M,N,K,w", WIDE_SHAPES)
def test_wide_items_accumulators_and_outputs_bit_exact(M, N, K, w):
    rng = np.random.default_rng(M + 7 * N + 11 * K + (0 if w is None else w))
    qa, qw = rand_codes(rng, (M, K)), rand_codes(rng, (N, K))
    s_tok = (rng.random(M) * 0.05 + 0.01).astype(np.float32)
    s_ch = (rng.random(N) * 0.0008 + 0.0002).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.01).astype(np.float32)
    ref = oracle.linear_fused_int8(qa, s_tok, qw, s_ch, bias)
    dev = [torch.from_numpy(a).to(DEV) for a in (qa, qw, s_tok, s_ch, bias)]
    wide_cfg = next(i for i in range(n_tc_configs()) if "2 x 256" in w8.config_name(i))
    w8.force_config(wide_cfg if w is None else wide_cfg + ((w + 1) << 12))
    ws = w8.alloc_workspace(M, N, K, w8.ACT_INT8, DEV)
    assert w8.int8_linear_plan(M, N, K, w8.ACT_INT8, ws.numel())["config"] == wide_cfg
    acc = w8.int8_gemm_i32_debug(dev[0], dev[1], ws)
    check_status(ws)
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    canvas = torch.full((M + 3, N + 24), -2.0, dtype=torch.bfloat16, device=DEV)     # guard band around the output
    out = canvas[1:1 + M, 8:8 + N]
    for _ in range(2):
        w8.int8_linear_fused(dev[0], dev[1], dev[3], dev[4], s_tok=dev[2], out=out, workspace=ws)
        check_status(ws)
        assert_bf16_close(synth.bf16_bits(out.contiguous().cpu()), ref["out"])
    mask = torch.ones_like(canvas, dtype=torch.bool)
    mask[1:1 + M, 8:8 + N] = False
    assert (canvas[mask] == -2.0).all()


# ------------------------------------------------------------------------------- banded tile order

@pytest.mark.parametrize("M,N,K,cfg,band", [(1300, 1288, 400, 2, 2), (1300, 1288, 400, 2, 3), (1300, 1288, 400, 2, 8),
                                             (700, 2056, 272, 0, 4), (520, 1032, 4096, 2, 2), (300, 520, 2064, 4, 5)])
def test_banded_tile_order_is_bit_exact(M, N, K, cfg, band):
    # bands of row blocks walked column by column (the order used when the operands exceed L2), forced on small
    # shapes: ragged last band, ragged edges, and a shape whose partial wave is cut along K
    rng = np.random.default_rng(M + 3 * N + 5 * K + band)
    qa, qw = rand_codes(rng, (M, K)), rand_codes(rng, (N, K))
    s_tok = (rng.random(M) * 0.05 + 0.01).astype(np.float32)
    s_ch = (rng.random(N) * 0.0008 + 0.0002).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.01).astype(np.float32)
    ref = oracle.linear_fused_int8(qa, s_tok, qw, s_ch, bias)
    dev = [torch.from_numpy(a).to(DEV) for a in (qa, qw, s_tok, s_ch, bias)]
    w8.force_config(cfg + (band << 20))
    ws = w8.alloc_workspace(M, N, K, w8.ACT_INT8, DEV)
    ws = torch.empty(ws.numel() + (16 << 20), dtype=torch.uint8, device=DEV)
    acc = w8.int8_gemm_i32_debug(dev[0], dev[1], ws)
    check_status(ws)
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    out = w8.int8_linear_fused(dev[0], dev[1], dev[3], dev[4], s_tok=dev[2], workspace=ws)
    check_status(ws)
    assert_bf16_close(synth.bf16_bits(out.cpu()), ref["out"])


# ------------------------------------------------------------------------------- random shapes, every configuration

def test_random_shapes_all_configurations_match_the_oracle():
    # 40 seeded random shapes (ragged in every dimension, K tails inside a pipeline stage, one to a few hundred
    # tiles). On every shape the oracle gives the accumulators and the output; the CUDA-core path and every
    # tensor-core configuration, with and without the K-split, must reproduce both bit for bit.
    rng = np.random.default_rng(2606)
    simt = n_tc_configs()
    big_ws = torch.empty(48 << 20, dtype=torch.uint8, device=DEV)
    for case in range(40):
        M = int(rng.integers(1, 700))
        N = 8 * int(rng.integers(1, 190))
        K = 16 * int(rng.integers(1, 380))
        qa, qw = rand_codes(rng, (M, K)), rand_codes(rng, (N, K))
        s_tok = (rng.random(M) * 0.05 + 0.01).astype(np.float32)
        s_ch = (rng.random(N) * 0.0008 + 0.0002).astype(np.float32)
        bias = (rng.standard_normal(N) * 0.01).astype(np.float32)
        dev = [torch.from_numpy(a).to(DEV) for a in (qa, qw, s_tok, s_ch, bias)]
        w8.force_config(simt)
        acc_ref = w8.int8_gemm_i32_debug(dev[0], dev[1], big_ws)
        out_ref = w8.int8_linear_fused(dev[0], dev[1], dev[3], dev[4], s_tok=dev[2], workspace=big_ws).clone()
        check_status(big_ws)
        ref = oracle.linear_fused_int8(qa, s_tok, qw, s_ch, bias)
        assert np.array_equal(acc_ref.cpu().numpy(), ref["acc"]), (M, N, K)
        assert_bf16_close(synth.bf16_bits(out_ref.cpu()), ref["out"])
        for cfg in range(simt):
            for forced in (cfg, cfg + 0x100):
                w8.force_config(forced)
                acc = w8.int8_gemm_i32_debug(dev[0], dev[1], big_ws)
                out = w8.int8_linear_fused(dev[0], dev[1], dev[3], dev[4], s_tok=dev[2], workspace=big_ws)
                check_status(big_ws)
                assert torch.equal(acc, acc_ref), (M, N, K, forced)
                assert torch.equal(out, out_ref), (M, N, K, forced)


# ------------------------------------------------------------------------------- two streams

def test_two_streams_with_their_own_workspaces_do_not_disturb_each_other():
    # calls on different streams may overlap on the device as long as each has its own workspace
    specs = [synth.LinearSpec("s0", 700, 1024, 1544), synth.LinearSpec("s1", 520, 8192, 776)]   # the second one is cut along K
    lanes = []
    for spec in specs:
        t = synth.make_linear(spec)
        qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
        A, bias = t["A"].to(DEV), t["bias"].to(DEV)
        ws = w8.alloc_workspace(spec.M, spec.N, spec.K, w8.ACT_BF16, DEV)
        want = w8.int8_linear_fused(A, qw, s_ch, bias, workspace=ws).clone()
        check_status(ws)
        lanes.append({"A": A, "qw": qw, "s_ch": s_ch, "bias": bias, "ws": ws, "want": want,
                      "out": torch.empty_like(want), "stream": torch.cuda.Stream(DEV)})
    torch.cuda.synchronize()
    for _ in range(25):
        for L in lanes:
            with torch.cuda.stream(L["stream"]):
                w8.int8_linear_fused(L["A"], L["qw"], L["s_ch"], L["bias"], out=L["out"], workspace=L["ws"])
    torch.cuda.synchronize()
    for L in lanes:
        check_status(L["ws"])
        assert torch.equal(L["out"], L["want"])


# ------------------------------------------------------------------------------- CUDA graph of a block's linears

def test_cuda_graph_replay_of_several_linears():
    # the calls allocate nothing and only enqueue work on the caller's stream, so a set of linears can be
    # captured once and replayed on new activations written into the same buffers
    shapes = [(300, 384, 328), (300, 320, 1024), (256, 8192, 264), (2, 384, 512)]   # plain, chained sizes, K-split, skinny
    layers = []
    for i, (M, K, N) in enumerate(shapes):
        spec = synth.LinearSpec(f"graph{i}", M, K, N)
        t = synth.make_linear(spec)
        qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(t["W"].numpy())
        qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
        layers.append({"spec": spec, "qw_ref": qw_ref, "s_ch_ref": s_ch_ref, "bias_np": t["bias"].numpy(),
                       "A": t["A"].to(DEV), "qw": qw, "s_ch": s_ch, "bias": t["bias"].to(DEV),
                       "out": torch.empty((M, N), dtype=torch.bfloat16, device=DEV),
                       "ws": w8.alloc_workspace(M, N, K, w8.ACT_BF16, DEV)})

    def run_all():
        for L in layers:
            w8.int8_linear_fused(L["A"], L["qw"], L["s_ch"], L["bias"], out=L["out"], workspace=L["ws"])

    run_all()                                           # first calls (one-time set-up) outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        run_all()
    for seed in (11, 12):
        for L in layers:
            L["A_new"] = synth.make_activations(L["spec"], seed)
            L["A"].copy_(L["A_new"].to(DEV))
            L["out"].fill_(-3.0)
        graph.replay()
        torch.cuda.synchronize()
        for L in layers:
            check_status(L["ws"])
            ref = oracle.linear_fused_bf16(synth.bf16_bits(L["A_new"]), L["qw_ref"], L["s_ch_ref"], L["bias_np"])
            assert_bf16_close(synth.bf16_bits(L["out"].cpu()), ref["out"])


# ------------------------------------------------------------------------------- benchmark configs, full size (T4)

ALL_SPECS = [s for name in ("c1", "c2", "c3", "c4", "c5", "paper") for s in synth.CONFIGS[name]]


@pytest.mark.parametrize("spec", ALL_SPECS, ids=[s.name for s in ALL_SPECS])
def test_benchmark_configs_full_size(spec):
    """The launch configuration bench.py times (automatic choice, from bf16), at full size, against the oracle
    on EVERY element: the oracle runs the whole linear (all rows, all columns: a minute and a half of host time
    for the sixteen linears together), and all int8 codes, all scales, all int32 accumulators and all bf16
    outputs of the CUDA path must equal its results bit for bit. The accumulators are also compared with the
    library integer matmul (the paper's own gate)."""
    t = synth.make_linear(spec)
    M, K, N = spec.M, spec.K, spec.N
    qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(t["W"].numpy())
    qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
    assert np.array_equal(qw.cpu().numpy(), qw_ref) and np.array_equal(s_ch.cpu().numpy(), s_ch_ref)
    A, bias = t["A"].to(DEV), t["bias"].to(DEV)
    ws = w8.alloc_workspace(M, N, K, w8.ACT_BF16, DEV)
    if spec.name in ("paper_ffn_down", "paper_llm_proj"):       # deep K and a nearly empty last wave: cut along K
        assert w8.int8_linear_plan(M, N, K, w8.ACT_BF16, ws.numel())["split_parts"] >= 2
    out = w8.int8_linear_fused(A, qw, s_ch, bias, workspace=ws)
    check_status(ws)
    ref = oracle.linear_fused_bf16(synth.bf16_bits(t["A"]), qw_ref, s_ch_ref, t["bias"].numpy())
    s_off, q_off = w8.int8_linear_workspace_offsets(M, K)
    s_tok = ws[s_off:s_off + 4 * M].view(torch.float32)
    qa = ws[q_off:q_off + M * K].view(torch.int8).view(M, K)
    assert np.array_equal(s_tok.cpu().numpy().view(np.uint32), ref["s_tok"].view(np.uint32))
    assert np.array_equal(qa.cpu().numpy(), ref["qa"])
    got = synth.bf16_bits(out.cpu())
    assert np.array_equal(got, ref["out"]), f"{int((got != ref['out']).sum())} of {got.size} outputs differ"
    assert_bf16_close(got, ref["out"])                  # the stated bar (1 ulp, relative error, cosine, finite)
    # raw accumulators of the same launch configuration: every element vs the oracle, and vs the library integer matmul
    ws_acc = w8.alloc_workspace(M, N, K, w8.ACT_INT8, DEV)
    acc = w8.int8_gemm_i32_debug(qa, qw, ws_acc)
    check_status(ws_acc)
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    if M > 16:
        assert torch.equal(acc, torch._int_mm(qa, qw.t()))
    # pre-quantized entry gives the same bits as the from-bf16 entry
    ws2 = w8.alloc_workspace(M, N, K, w8.ACT_INT8, DEV)
    out2 = w8.int8_linear_fused(qa, qw, s_ch, bias, s_tok=s_tok, workspace=ws2)
    check_status(ws2)
    assert torch.equal(out2, out)


# ------------------------------------------------------------------------------- more than 2^31 elements

def test_quantizer_beyond_two_to_the_31_elements():
    # 41 repeats of a 1000-row block of 104 KB rows: 2.18e9 activations. Every repeat must carry the codes the oracle
    # gives for the block (an index that wrapped at 2^31 would read or write the wrong rows).
    K, rows, reps = 53248, 1000, 41
    assert rows * reps * K > 2 ** 31
    block = synth.make_activations(synth.LinearSpec("big_q", rows, K, 8))
    qa_ref, s_ref = oracle.quantize_act_per_token(synth.bf16_bits(block))
    A = block.to(DEV).repeat(reps, 1)
    qa, s = w8.int8_quantize_act_per_token(A)
    del A
    qa_ref_d, s_ref_d = torch.from_numpy(qa_ref).to(DEV), torch.from_numpy(s_ref).to(DEV)
    assert torch.equal(s.view(reps, rows), s_ref_d.expand(reps, rows))
    for r in range(reps):
        assert torch.equal(qa[r * rows:(r + 1) * rows], qa_ref_d), r


def test_fused_output_beyond_two_to_the_31_elements():
    # 46400 x 46400 outputs (2.15e9, 4.3 GB of bf16) from a short K: the activation rows repeat a 928-row block, so
    # every block of output rows must equal the oracle's result for that block.
    M, N, K, rows = 46400, 46400, 64, 928
    assert M * N > 2 ** 31 and M % rows == 0
    rng = np.random.default_rng(31)
    qa_b, qw = rand_codes(rng, (rows, K)), rand_codes(rng, (N, K))
    s_tok_b = (rng.random(rows) * 0.05 + 0.01).astype(np.float32)
    s_ch = (rng.random(N) * 0.0008 + 0.0002).astype(np.float32)
    bias = (rng.standard_normal(N) * 0.01).astype(np.float32)
    ref = torch.from_numpy(oracle.linear_fused_int8(qa_b, s_tok_b, qw, s_ch, bias)["out"].view(np.int16)).to(DEV)
    reps = M // rows
    qa = torch.from_numpy(qa_b).to(DEV).repeat(reps, 1)
    s_tok = torch.from_numpy(s_tok_b).to(DEV).repeat(reps)
    ws = w8.alloc_workspace(M, N, K, w8.ACT_INT8, DEV)
    out = w8.int8_linear_fused(qa, torch.from_numpy(qw).to(DEV), torch.from_numpy(s_ch).to(DEV), torch.from_numpy(bias).to(DEV),
                               s_tok=s_tok, workspace=ws)
    check_status(ws)
    got = out.view(torch.int16)
    for r in range(reps):
        assert torch.equal(got[r * rows:(r + 1) * rows], ref), r


# ------------------------------------------------------------------------------- bounded waits that run out

@pytest.fixture
def short_waits():
    """Device-side waits of a few milliseconds instead of 2 s, and the starvation hook reset afterwards."""
    old = w8.debug_set_wait_limit_ns(3_000_000)
    yield
    w8.debug_set_starve(0)
    w8.debug_set_wait_limit_ns(old)
    torch.cuda.synchronize()
    w8.int8_sticky_status(clear=True)


def _timeout_case(M, K, N, seed=0):
    spec = synth.LinearSpec(f"to{M}x{K}x{N}", M, K, N)
    t = synth.make_linear(spec, seed)
    qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(t["W"].numpy())
    ref = oracle.linear_fused_bf16(synth.bf16_bits(t["A"]), qw_ref, s_ch_ref, t["bias"].numpy())
    qw, s_ch = w8.int8_quantize_weight_per_channel(t["W"].to(DEV))
    return spec, t["A"].to(DEV), qw, s_ch, t["bias"].to(DEV), ref


# one CTA per tile / a CTA pair / a pair of two sub-tiles / a shape that is cut along K
@pytest.mark.parametrize("M,K,N,cfg", [(128, 512, 256, 0), (300, 1024, 520, 2), (300, 1024, 520, 5), (256, 8192, 256, 2)])
def test_gemm_wait_runs_out_and_the_kernel_returns(short_waits, M, K, N, cfg):
    """The producer withholds one pipeline stage (nothing invalid is touched): the MMA thread's wait on it runs
    out after 3 ms, every role of every CTA unwinds, TMEM is freed, the kernel returns and the status word says
    so. The next, normal call on the same workspace must be bit-exact again."""
    spec, A, qw, s_ch, bias, ref = _timeout_case(M, K, N)
    w8.force_config(cfg)
    ws = w8.alloc_workspace(M, N, K, w8.ACT_BF16, DEV)
    if K == 8192:
        assert w8.int8_linear_plan(M, N, K, w8.ACT_BF16, ws.numel())["split_parts"] >= 2
    w8.int8_sticky_status(clear=True)
    w8.debug_set_starve(1)
    out = w8.int8_linear_fused(A, qw, s_ch, bias, workspace=ws)
    w8.debug_set_starve(0)
    torch.cuda.synchronize()                          # returns: the kernel did not hang
    raw_word = int(ws[:4].view(torch.int32).item())
    assert raw_word & 0xff == 7 and (raw_word >> 8) in (1, 2, 3, 4), hex(raw_word)     # TIMEOUT, and which wait gave up
    assert w8.int8_check_status(ws) == 7              # W8A8_ERR_TIMEOUT, then cleared
    assert w8.int8_check_status(ws) == 0
    # a later call on the same workspace resets the word, the sticky word keeps the time-out until it is read
    out = w8.int8_linear_fused(A, qw, s_ch, bias, workspace=ws)
    assert w8.int8_check_status(ws) == 0
    assert_bf16_close(synth.bf16_bits(out.cpu()), ref["out"])
    assert w8.int8_sticky_status(clear=True) == 7
    assert w8.int8_sticky_status(clear=True) == 0


# row-slot barriers fed by 16 lanes / by one lane, one-row stages, and stage barriers (two CTAs per SM, rows above 4 KB)
@pytest.mark.parametrize("M,K", [(300, 1024), (40, 12288), (6, 53248), (9481, 3072)])
def test_quantizer_wait_runs_out_and_the_kernel_returns(short_waits, M, K):
    spec = synth.LinearSpec(f"toq{M}x{K}", M, K, 8)
    A = synth.make_activations(spec)
    qa_ref, s_ref = oracle.quantize_act_per_token(synth.bf16_bits(A))
    dA = A.to(DEV)
    w8.int8_sticky_status(clear=True)
    w8.debug_set_starve(2)
    w8.int8_quantize_act_per_token(dA)
    w8.debug_set_starve(0)
    torch.cuda.synchronize()
    assert w8.int8_sticky_status(clear=True) == 7     # the standalone quantizer has no workspace: only the sticky word tells
    qa, s = w8.int8_quantize_act_per_token(dA)
    assert np.array_equal(qa.cpu().numpy(), qa_ref) and np.array_equal(s.cpu().numpy(), s_ref)
    assert w8.int8_sticky_status(clear=True) == 0
    # and inside the fused call: the quantizer's time-out lands in the workspace status word
    N = 264
    W = synth.make_weight(synth.LinearSpec(f"toqw{K}", M, K, N))
    qw, s_ch = w8.int8_quantize_weight_per_channel(W.to(DEV))
    ws = w8.alloc_workspace(M, N, K, w8.ACT_BF16, DEV)
    w8.debug_set_starve(2)
    w8.int8_linear_fused(dA, qw, s_ch, None, workspace=ws)
    w8.debug_set_starve(0)
    assert w8.int8_check_status(ws) == 7
    out = w8.int8_linear_fused(dA, qw, s_ch, None, workspace=ws)
    assert w8.int8_check_status(ws) == 0
    qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(W.numpy())
    ref = oracle.linear_fused_bf16(synth.bf16_bits(A), qw_ref, s_ch_ref, None)
    assert_bf16_close(synth.bf16_bits(out.cpu()), ref["out"])
    assert w8.int8_sticky_status(clear=True) == 7


# ------------------------------------------------------------------------------- one-kernel path for small problems

@pytest.fixture
def small_path():
    """Yields a setter of the one-kernel path's mode; the default (chosen from the shape) is restored afterwards."""
    yield w8.debug_set_small_path
    w8.debug_set_small_path(-1)


# K <= 256 / 512 / 1024 (one, two, four 16-byte units per lane) x clusters of 1, 2 and 4 CTAs (N <= 32, <= 64, more),
# ragged M, N and K, a grid padded to whole clusters (N = 264: 9 CTAs -> 12), a single token, the largest shape
@pytest.mark.parametrize("M,K,N", [(128, 256, 256), (100, 272, 264), (9, 16, 8), (77, 1008, 40), (1, 512, 96),
                                   (128, 1024, 1024), (33, 640, 2048), (128, 128, 32), (64, 768, 4736), (17, 48, 56)])
def test_one_kernel_path_against_oracle(small_path, M, K, N):
    rng = np.random.default_rng(M * 7 + K + N)
    A = torch.from_numpy(rng.standard_normal((M, K), dtype=np.float32)).to(torch.bfloat16)
    if M > 2:
        A[1] = 0                                   # an all-zero token
    W = rng.standard_normal((N, K), dtype=np.float32) * np.float32(0.02)
    bias = rng.standard_normal(N, dtype=np.float32) * np.float32(0.01)
    qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(W)
    bits = synth.bf16_bits(A)
    ref = oracle.linear_fused_bf16(bits, qw_ref, s_ch_ref, bias)
    ref_nb = oracle.linear_fused_bf16(bits, qw_ref, s_ch_ref, None)
    # activations as a view with a row stride, output into a wider buffer
    A_wide = torch.zeros((M, K + 32), dtype=torch.bfloat16, device=DEV)
    A_wide[:, :K] = A.to(DEV)
    dA = A_wide[:, :K]
    out_wide = torch.full((M, N + 16), 7.0, dtype=torch.bfloat16, device=DEV)
    qw, s_ch = w8.int8_quantize_weight_per_channel(torch.from_numpy(W).to(DEV))
    db = torch.from_numpy(bias).to(DEV)
    ws = w8.alloc_workspace(M, N, K, w8.ACT_BF16, DEV)
    small_path(1)
    assert "one kernel" in w8.int8_linear_plan(M, N, K, w8.ACT_BF16, ws.numel())["name"]
    ws.zero_()
    out, rowmax = w8.int8_linear_fused_rowmax(dA, qw, s_ch, db, out=out_wide[:, :N], workspace=ws)
    check_status(ws)
    assert np.array_equal(synth.bf16_bits(out.cpu()), ref["out"])
    assert torch.all(out_wide[:, N:] == 7.0)       # nothing written beyond the N columns
    assert np.array_equal(rowmax.cpu().numpy(), oracle.row_absmax_bf16(ref["out"]))
    # the workspace holds codes and scales, as after the two-kernel path
    s_off, q_off = w8.int8_linear_workspace_offsets(M, K)
    assert np.array_equal(ws[q_off:q_off + M * K].view(torch.int8).view(M, K).cpu().numpy(), ref["qa"])
    assert np.array_equal(ws[s_off:s_off + 4 * M].view(torch.float32).cpu().numpy().view(np.uint32), ref["s_tok"].view(np.uint32))
    # without bias; with the absmax of every row handed in (one-pass quantizer inside the kernel)
    out_nb = w8.int8_linear_fused(dA, qw, s_ch, None, workspace=ws)
    check_status(ws)
    assert np.array_equal(synth.bf16_bits(out_nb.cpu()), ref_nb["out"])
    amax = torch.from_numpy(oracle.row_absmax_bf16(bits)).to(DEV)
    out_g, _ = w8.int8_linear_fused_rowmax(dA, qw, s_ch, db, workspace=ws, rowmax_in=amax)
    check_status(ws)
    assert np.array_equal(synth.bf16_bits(out_g.cpu()), ref["out"])
    # and the two-kernel path gives the same bits on the same call
    small_path(0)
    assert "one kernel" not in w8.int8_linear_plan(M, N, K, w8.ACT_BF16, ws.numel())["name"]
    out2 = w8.int8_linear_fused(dA, qw, s_ch, db, workspace=ws)
    check_status(ws)
    assert np.array_equal(synth.bf16_bits(out2.cpu()), ref["out"])
    assert w8.int8_sticky_status(clear=True) == 0


def test_one_kernel_path_wait_runs_out_and_the_kernel_returns(short_waits, small_path):
    """The MMA thread never commits (nothing invalid is touched): the epilogue warps' wait runs out after 3 ms, TMEM is
    freed, the kernel returns and the status word says so; the next call on the same workspace is exact again."""
    M, K, N = 128, 256, 256
    spec, A, qw, s_ch, bias, ref = _timeout_case(M, K, N)
    ws = w8.alloc_workspace(M, N, K, w8.ACT_BF16, DEV)
    small_path(1)
    w8.int8_sticky_status(clear=True)
    w8.debug_set_starve(1)
    w8.int8_linear_fused(A, qw, s_ch, bias, workspace=ws)
    w8.debug_set_starve(0)
    torch.cuda.synchronize()                          # returns: the kernel did not hang
    raw_word = int(ws[:4].view(torch.int32).item())
    assert raw_word & 0xff == 7 and (raw_word >> 8) == 4, hex(raw_word)
    assert w8.int8_check_status(ws) == 7
    out = w8.int8_linear_fused(A, qw, s_ch, bias, workspace=ws)
    assert w8.int8_check_status(ws) == 0
    assert np.array_equal(synth.bf16_bits(out.cpu()), ref["out"])
    assert w8.int8_sticky_status(clear=True) == 7
    assert w8.int8_sticky_status(clear=True) == 0


def test_one_kernel_path_random_small_shapes(small_path):
    """200 seeded random shapes (M <= 128, K <= 1024, N <= 2400, with and without bias, an all-zero token) through the
    one-kernel path: output, row maxima and the codes left in the workspace against the oracle, bit for bit."""
    small_path(1)
    for seed in range(200):
        rng = np.random.default_rng(9000 + seed)
        M, K, N = int(rng.integers(1, 129)), 16 * int(rng.integers(1, 65)), 8 * int(rng.integers(1, 300))
        A = torch.from_numpy(rng.standard_normal((M, K), dtype=np.float32) * np.float32(rng.choice([0.05, 1.0, 30.0]))).to(torch.bfloat16)
        if M > 3:
            A[int(rng.integers(0, M))] = 0
        W = rng.standard_normal((N, K), dtype=np.float32) * np.float32(0.02)
        bias = rng.standard_normal(N, dtype=np.float32) * np.float32(0.01) if rng.integers(0, 2) else None
        qw_ref, s_ch_ref = oracle.quantize_weight_per_channel(W)
        ref = oracle.linear_fused_bf16(synth.bf16_bits(A), qw_ref, s_ch_ref, bias)
        qw, s_ch = w8.int8_quantize_weight_per_channel(torch.from_numpy(W).to(DEV))
        ws = w8.alloc_workspace(M, N, K, w8.ACT_BF16, DEV)
        out, rowmax = w8.int8_linear_fused_rowmax(A.to(DEV), qw, s_ch, None if bias is None else torch.from_numpy(bias).to(DEV), workspace=ws)
        check_status(ws)
        assert np.array_equal(synth.bf16_bits(out.cpu()), ref["out"]), (M, K, N)
        assert np.array_equal(rowmax.cpu().numpy(), oracle.row_absmax_bf16(ref["out"])), (M, K, N)
        s_off, q_off = w8.int8_linear_workspace_offsets(M, K)
        assert np.array_equal(ws[q_off:q_off + M * K].view(torch.int8).view(M, K).cpu().numpy(), ref["qa"]), (M, K, N)
    assert w8.int8_sticky_status(clear=True) == 0
