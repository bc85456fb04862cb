"""World-size-2 CPU (gloo) test of the benchmark's multi-rank plumbing: row sharding covers the tokens
exactly once, and whole-job throughput is all ranks' units over the slowest rank's time."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import numpy as np
    import oracle
    from paper_2606_14598_b200 import dist as wdist
    from paper_2606_14598_b200 import inputs as synth
    rank, local_rank, world = wdist.init("gloo")
    spec = synth.LinearSpec("gloo", 50, 64, 24)
    lo, hi = wdist.shard_rows(spec.M, rank, world, multiple=8)
    # each rank runs the (row-local) path on its own rows; weights are replicated
    t = synth.make_linear(spec)
    qw, s_ch = oracle.quantize_weight_per_channel(t["W"].numpy())
    A = np.ascontiguousarray(synth.bf16_bits(t["A"])[lo:hi])
    part = oracle.linear_fused_bf16(A, qw, s_ch, t["bias"].numpy())["out"]
    full = oracle.linear_fused_bf16(synth.bf16_bits(t["A"]), qw, s_ch, t["bias"].numpy())["out"]
    same = bool((part == full[lo:hi]).all())
    wdist.barrier()
    value, tmax = wdist.aggregate_throughput(float(hi - lo), 1.0 + rank)
    rows_total = wdist.sum_over_ranks(float(hi - lo))
    print(json.dumps({"rank": rank, "lo": lo, "hi": hi, "same": same, "value": value, "tmax": tmax, "rows": rows_total}))
""") % ROOT


def test_two_ranks_gloo():
    # the ranks meet through a rendezvous file (no port is picked ahead of time, so no other process can take it)
    import json
    from paper_2606_14598_b200.dist import spawn_ranks
    results = spawn_ranks([sys.executable, "-c", WORKER], 2, extra_env={"OMP_NUM_THREADS": "2"}, timeout=180)
    outs = []
    for rc, o, e in results:
        assert rc == 0, e[-2000:]
        outs.append(json.loads(o.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    assert outs[0]["lo"] == 0 and outs[0]["hi"] == outs[1]["lo"] and outs[1]["hi"] == 50
    assert all(d["same"] for d in outs)                      # sharding over tokens changes no bits
    assert all(d["rows"] == 50.0 and d["tmax"] == 2.0 and d["value"] == 25.0 for d in outs)


def _run_two_ranks_on_a_port():
    import json
    import socket
    s = socket.socket()
    s.setsockopt(socket.SOL_SOCKET, socket.SO_REUSEADDR, 1)
    s.bind(("127.0.0.1", 0))
    port = str(s.getsockname()[1])
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=port,
                   OMP_NUM_THREADS="2")
        env.pop("W8A8_RDZV_FILE", None)
        if r == 0:
            s.close()
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs, errs = [], []
    for p in procs:
        o, e = p.communicate(timeout=180)
        errs.append(e)
        if p.returncode != 0:
            return None, errs
        outs.append(json.loads(o.strip().splitlines()[-1]))
    return outs, errs


def test_two_ranks_gloo_through_master_addr_and_port():
    # the launcher's way (torchrun sets MASTER_ADDR / MASTER_PORT): rank 0 opens the store on a port this test asked
    # the kernel for and held open with SO_REUSEADDR until the ranks start. Another process can still take the port in
    # the moment between close and bind, so one failed rendezvous is retried on a new port.
    outs, errs = _run_two_ranks_on_a_port()
    if outs is None:
        outs, errs = _run_two_ranks_on_a_port()
    assert outs is not None, errs[0][-2000:]
    assert all(d["same"] and d["rows"] == 50.0 for d in outs)


def test_shard_rows_partition():
    from paper_2606_14598_b200.dist import shard_rows
    for M in (1, 2, 50, 4608, 9216, 4609):
        for world in (1, 2, 3, 8):
            for mult in (1, 128):
                spans = [shard_rows(M, r, world, mult) for r in range(world)]
                assert spans[0][0] == 0 and spans[-1][1] == M
                assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
                sizes = [hi - lo for lo, hi in spans]
                assert max(sizes) - min(sizes) <= 2 * mult - 1


def test_reference_arm_prints_one_json_line_and_only_on_rank_zero():
    # `bench.py --impl reference` times the CPU oracle and needs no GPU; launched as ranks of a multi-process job,
    # rank 0 alone does the work and prints, the others leave at once
    import json
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1", "--steps", "1", "--warmup", "0"]
    env = dict(os.environ, OMP_NUM_THREADS="2")
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        env.pop(k, None)
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "TOPS" and d["value"] > 0 and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["sample"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0 and d["gpu_launches"] == 0
    assert d["config"]["workload"].startswith("c1")
    env1 = dict(env, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    r1 = subprocess.run(cmd + ["--gpus", "2"], env=env1, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r1.returncode == 0 and r1.stdout.strip() == "", r1.stderr[-2000:]
    # without a launcher `--gpus 2` starts the two ranks itself: still exactly one line, from rank 0
    r2 = subprocess.run(cmd + ["--gpus", "2"], env=env, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r2.returncode == 0, r2.stderr[-2000:]
    lines2 = [ln for ln in r2.stdout.splitlines() if ln.strip()]
    assert len(lines2) == 1 and json.loads(lines2[0])["n_gpus"] == 2 and json.loads(lines2[0])["impl"] == "reference"
    # the reference arm times exactly --steps steps after --warmup untimed ones
    r3 = subprocess.run(cmd[:-4] + ["--steps", "4", "--warmup", "2"], env=env, capture_output=True, text=True, timeout=300, cwd=ROOT)
    d3 = json.loads(r3.stdout.strip().splitlines()[-1])
    assert d3["steps"] == 4 and d3["warmup"] == 2
