#!/usr/bin/env python
"""Benchmark of the fused W8A8 linear on seeded synthetic DiT-shaped inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl reference]

One step = one pass of the whole hot path (per-token quantization of the bf16 activations, int8
tensor-core GEMM, dequantizing epilogue) over every linear of the workload; the default workload
is the MLP up and down projections at 1024px (M=4608, 3072 -> 12288 -> 3072), the shapes the
throughput target is quoted on. Prints ONE JSON line on stdout (diagnostics go to stderr).

`--impl reference` times the CPU oracle, as it stands, on the host cores on a bounded sample of
the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused W8A8 linear TOPS (% of B200 dense INT8 peak) per DiT GEMM shape"
INT8_PEAK_TOPS = 4500.0            # B200 datasheet, dense INT8
# DRAM traffic of one gemm_tc_kernel launch (dram__bytes_read.sum + dram__bytes_write.sum of an ncu capture of this
# program on that workload, averaged over the workload's GEMM launches), with the summary it is taken from. Workloads
# that were not captured have no entry: the bench line then says null and why.
NCU_GEMM_DRAM_TRAFFIC = {
    "c4": {"bytes_per_launch": 126.3e6, "profile": "profiles/gemm_tc_kernel_c4_mlp.md",
           "note": "mean of the up (124.8 MB) and down (127.7 MB) launches; algorithmic bytes 165.2 / 122.7 MB"},
    "paper": {"bytes_per_launch": None, "profile": "profiles/gemm_tc_kernel_paper_llm_proj_ksplit.md",
              "note": "only the llm-proj launch was captured (1.42 GB against 502 MB algorithmic); no per-workload mean"},
}
L2_BYTES = 126 * 1024 * 1024


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------ clocks

SAMPLER_SRC = r"""
import json, sys, time
idx, period = sys.argv[1], float(sys.argv[2])
sys.stdout = open(sys.argv[3], "a", buffering=1)
import pynvml as nv
nv.nvmlInit()
h = nv.nvmlDeviceGetHandleByIndex(int(idx)) if idx.isdigit() else nv.nvmlDeviceGetHandleByUUID(idx)
print(json.dumps({"max_mhz": float(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))}), flush=True)
pw, mask, n = None, 0, 0
while True:
    t = time.time()
    try:
        mhz = float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
        if n % 4 == 0:      # the clock every round; power and clock-event reasons (slower queries) every fourth
            pw = nv.nvmlDeviceGetPowerUsage(h) / 1000.0
            try:
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
            except Exception:
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
        n += 1
        sys.stdout.write(json.dumps({"t": t, "mhz": mhz, "w": pw, "mask": int(mask), "dt": time.time() - t}) + "\n")
        sys.stdout.flush()
    except Exception:
        pass
    time.sleep(period)
"""


class ClockSampler:
    """Samples SM clock, power and clock-event reasons through NVML while the timed region runs. The sampling loop is
    a process of its own (a thread of this one is starved by the launch loop), started ahead of the warm-up; only the
    samples whose time stamps fall between enter and exit are kept."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x100: "display_clock_setting",
               0x10: "sync_boost"}

    def __init__(self, index: int, period_s: float = 0.001):
        import subprocess
        self.samples, self.power, self.reasons, self.times = [], [], set(), []
        self.max_mhz, self.t0, self.t1, self.proc, self.out = None, None, None, None, None
        visible = os.environ.get("CUDA_VISIBLE_DEVICES")
        tok = str(index)
        if visible:
            ids = [v for v in visible.split(",") if v.strip() != ""]
            tok = ids[index] if index < len(ids) else ids[0]
        try:
            # the samples go to a temporary file: a pipe would fill up (64 KB, a second or two of samples)
            # while nobody reads it and block the sampler for the rest of the run
            import tempfile
            fd, self.out = tempfile.mkstemp(prefix="w8a8_clocks_", suffix=".jsonl")
            os.close(fd)
            self.proc = subprocess.Popen([sys.executable, "-c", SAMPLER_SRC, tok, str(period_s), self.out],
                                         stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
            first, deadline = "", time.time() + 20.0
            while time.time() < deadline and self.proc.poll() is None:      # up once it has printed the maximum clock
                with open(self.out) as f:
                    first = f.readline()
                if first.endswith("\n"):
                    break
                time.sleep(0.02)
            self.max_mhz = json.loads(first)["max_mhz"] if first.endswith("\n") else None
            if self.max_mhz is None:
                raise RuntimeError("no answer from the sampler")
        except Exception as e:          # NVML missing: report that no clocks were sampled
            log(f"[bench] NVML sampler unavailable: {e}")
            self.close()

    def close(self):
        if self.proc is not None:
            self.proc.kill()
            self.proc.wait()
            self.proc = None
        if self.out is not None:
            try:
                os.unlink(self.out)
            except OSError:
                pass
            self.out = None

    def __enter__(self):
        self.t0 = time.time()
        return self

    def __exit__(self, *exc):
        self.t1 = time.time()
        if self.proc is None:
            return
        time.sleep(0.01)
        self.proc.kill()
        self.proc.wait()
        self.proc = None
        with open(self.out) as f:
            lines = f.read().splitlines()
        self.close()
        for ln in lines:
            try:
                d = json.loads(ln)
            except Exception:
                continue
            if "t" in d and self.t0 <= d["t"] <= self.t1:
                self.samples.append(d["mhz"])
                self.times.append(d["t"])
                if d["w"] is not None:
                    self.power.append(d["w"])
                for bit, name in self.REASONS.items():
                    if d["mask"] & bit:
                        self.reasons.add(name)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["not sampled"], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "sample_period_ms": (self.times[-1] - self.times[0]) / (len(self.times) - 1) * 1e3 if len(self.times) > 1 else None,
                "power_w_max": max(self.power) if self.power else None}


# ------------------------------------------------------------------------------------------ reference arm

def reference_sample_rows(spec, target_gmac=40.0):
    """Rows of one linear the oracle recomputes per step, sized for a few seconds of CPU work."""
    rows = int(target_gmac * 1e9 / (spec.K * spec.N))
    return max(1, min(spec.M, rows))


def time_oracle(specs, steps, warmup, target_gmac):
    """Times the oracle (quantize + integer GEMM + epilogue) on the first rows of each linear."""
    import numpy as np

    import oracle
    from paper_2606_14598_b200 import inputs as synth

    prepared = []
    for spec in specs:
        rows = reference_sample_rows(spec, target_gmac)
        A = synth.bf16_bits(synth.make_activations(spec, rows=slice(0, rows)))
        qw, s_ch = oracle.quantize_weight_per_channel(synth.make_weight(spec).numpy())
        bias = synth.make_bias(spec)
        prepared.append((spec, rows, np.ascontiguousarray(A), qw, s_ch, None if bias is None else bias.numpy()))
    ops = sum(2.0 * rows * s.N * s.K for s, rows, *_ in prepared)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        for _, _, A, qw, s_ch, bias in prepared:
            oracle.linear_fused_bf16(A, qw, s_ch, bias)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    sec = sum(times) / len(times)
    sample = ", ".join(f"{s.name}: first {rows} of {s.M} rows" for s, rows, *_ in prepared)
    return ops / sec / 1e12, sec, oracle.num_threads(), sample


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2606_14598_b200 import inputs as synth
    specs = workload_specs(args)
    # exactly --steps timed steps after --warmup untimed ones; a step is a bounded sample of the workload (the first
    # rows of every linear), sized so that the whole run takes about a minute of host time at ~40 GMAC/s
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    per_linear_gmac = max(0.05, min(20.0, 2400.0 / (steps + warmup))) / max(1, len(specs))
    tops, sec, cores, sample = time_oracle(specs, steps, warmup, target_gmac=per_linear_gmac)
    line = {
        "impl": "reference", "metric": METRIC, "value": tops, "unit": "TOPS", "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": workload_name(args.workload, specs), "sample": sample},
        "pct_of_int8_peak": 100.0 * tops / INT8_PEAK_TOPS,
        "cpu_baseline": {"value": tops, "unit": "TOPS", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tops, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_name(key, specs):
    return f"{key}: " + " + ".join(f"{s.name} (M={s.M}, K={s.K}, N={s.N})" for s in specs)


# ------------------------------------------------------------------------------------------ CUDA arm

def workload_specs(args):
    """The linears of the chosen workload, with the token count overridden if asked (skinny linears keep theirs)."""
    import dataclasses

    from paper_2606_14598_b200 import inputs as synth
    specs = synth.CONFIGS[args.workload]
    if args.rows > 0:
        specs = [s if s.M <= 16 else dataclasses.replace(s, M=args.rows, name=f"{s.name}_m{args.rows}") for s in specs]
    return specs


def cuda_timer(torch, fn, iters, warm):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for a, b in ev:
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) * 1e-3 for a, b in ev]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="c4", choices=["c1", "c2", "c3", "c4", "c5", "paper"])
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--sets", type=int, default=3, help="rotating input/weight sets (keeps steps out of L2)")
    ap.add_argument("--no-extras", action="store_true", help="skip e2e, context and CPU-baseline legs")
    ap.add_argument("--rows", type=int, default=0,
                    help="override the token count M of every linear of the workload (the paper sweeps M = 512 ... 16384)")
    ap.add_argument("--launch", default="direct", choices=["graph", "direct"],
                    help="graph: each step is one replay of a captured CUDA graph of the step's calls; direct: the calls themselves")
    ap.add_argument("--config", type=int, default=-1, help="force a kernel configuration (sweeps); -1 = from the shape")
    ap.add_argument("--repeats", type=int, default=0,
                    help="timed loops of --steps steps (0 = 7, enough for ten NVML samples over 20-step loops); the median is reported")
    ap.add_argument("--small-path", default="auto", choices=["auto", "on", "off"],
                    help="the one-kernel path for small problems: chosen from the shape / wherever it can run / never")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher: run one process per GPU ourselves (rank i on GPU i); the ranks meet through a rendezvous file
        from paper_2606_14598_b200 import dist as wdist
        results = wdist.spawn_ranks([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus)
        for r, (rc, out, err) in enumerate(results):
            sys.stderr.write(err)
            if r == 0:
                sys.stdout.write(out)
        sys.stdout.flush()
        raise SystemExit(max(rc for rc, _, _ in results))
    if args.impl == "reference":
        return run_reference(args)

    import torch

    import paper_2606_14598_b200 as w8
    from paper_2606_14598_b200 import dist as wdist
    from paper_2606_14598_b200 import inputs as synth
    from paper_2606_14598_b200 import roofline as model

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA path has no CPU fallback (use --impl reference)")
    args.warmup = max(args.warmup, 3)
    rank, local_rank, world = wdist.init("nccl")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    specs = workload_specs(args)
    peaks = measured_peaks()
    w8.force_config(args.config)
    w8.debug_set_small_path({"auto": -1, "on": 1, "off": 0}[args.small_path])

    # ---- set-up (untimed): seeded inputs, weights quantized on the device by the library
    sets = []
    for r in range(args.sets):
        layer = []
        for spec in specs:
            seed = 1000 * rank + r
            A = synth.make_activations(spec, seed).to(dev)
            qw, s_ch = w8.int8_quantize_weight_per_channel(synth.make_weight(spec, seed).to(dev))
            bias = synth.make_bias(spec, seed)
            layer.append({"spec": spec, "A": A, "qw": qw, "s_ch": s_ch, "bias": None if bias is None else bias.to(dev),
                          "out": torch.empty((spec.M, spec.N), dtype=torch.bfloat16, device=dev),
                          "ws": w8.alloc_workspace(spec.M, spec.N, spec.K, w8.ACT_BF16, dev)})
        sets.append(layer)
    torch.cuda.synchronize()
    set_bytes = sum(model.bytes_from_bf16(s.M, s.N, s.K) for s in specs)
    ops_per_step = float(sum(s.ops for s in specs))

    # the timed loop calls the C ABI directly with arguments marshalled once (keeps the host ahead of the GPU)
    from paper_2606_14598_b200 import binding
    raw = binding.raw()
    stream = torch.cuda.current_stream(dev).cuda_stream

    def fused_args(L, bf16=True, s_tok=None, qa=None, ws=None):
        sp = L["spec"]
        A = L["A"] if bf16 else qa
        ws = L["ws"] if ws is None else ws
        return (A.data_ptr(), 0 if bf16 else 1, sp.K, None if bf16 else s_tok.data_ptr(), L["qw"].data_ptr(),
                L["s_ch"].data_ptr(), None if L["bias"] is None else L["bias"].data_ptr(), L["out"].data_ptr(), sp.N,
                sp.M, sp.N, sp.K, ws.data_ptr(), ws.numel(), stream)

    step_args = [[fused_args(L) for L in layer] for layer in sets]

    def step(i):
        for a in step_args[i % len(step_args)]:
            rc = raw.int8_linear_fused(*a)
            if rc != 0:
                raise SystemExit(f"int8_linear_fused: {w8.status_string(rc)}")

    # ---- health gate: the GPU must deliver its usual bf16 rate, or the numbers below mean nothing
    health = None
    if rank == 0 and not args.no_extras:
        a = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
        b = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
        ts = cuda_timer(torch, lambda: torch.matmul(a, b), 10, 3)
        tf = 2 * 8192 ** 3 / min(ts) / 1e12
        health = {"bf16_matmul_tflops": tf, "ok": tf >= 0.8 * peaks["bf16_tflops"]}
        del a, b

    # ---- the timed region
    clocks = ClockSampler(local_rank)                      # its process starts now and samples through the warm-up too
    for i in range(max(args.warmup, len(step_args))):      # direct calls first: one-time set-up happens outside any capture
        step(i)
    torch.cuda.synchronize()
    graphs, launch_note = None, "direct calls of int8_linear_fused"
    if args.launch == "graph":
        # One CUDA graph per rotating set holds the calls of a step (they allocate nothing and only enqueue on the
        # stream they are given); the timed loop replays them, so no per-call host work sits between the kernels.
        try:
            graphs = []
            for i in range(len(step_args)):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    gs = torch.cuda.current_stream(dev).cuda_stream
                    for a_ in step_args[i]:
                        rc = raw.int8_linear_fused(*(a_[:-1] + (gs,)))
                        if rc != 0:
                            raise RuntimeError(w8.status_string(rc))
                graphs.append(g)
            launch_note = "one captured CUDA graph per rotating set (the step's int8_linear_fused calls), replayed"
        except Exception as ex:                              # noqa: BLE001 - report and time the calls themselves
            graphs, launch_note = None, f"direct calls of int8_linear_fused (graph capture failed: {ex})"

    def run_step(i):
        if graphs is not None:
            graphs[i % len(graphs)].replay()
        else:
            step(i)

    for i in range(max(3, args.warmup)):
        run_step(i)
    torch.cuda.synchronize()
    # a short burst first (rank 0's own figure, before the power cap engages some tens of milliseconds into a loop):
    # reported beside the headline, which is the long loop below
    burst = None
    if args.steps > 200:
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record()
        for i in range(100):
            run_step(i)
        b1.record()
        torch.cuda.synchronize()
        b_sec = b0.elapsed_time(b1) * 1e-3 / 100
        burst = {"value": ops_per_step / b_sec / 1e12, "unit": "TOPS", "ms_per_step": b_sec * 1e3, "steps": 100,
                 "pct_of_int8_peak": 100.0 * ops_per_step / b_sec / 1e12 / INT8_PEAK_TOPS,
                 "note": "this rank's first 100 steps after warm-up, before the power cap engages"}
    # R timed loops of exactly --steps steps each, every one bracketed by a barrier and a device synchronize on both
    # sides and timed with CUDA events on the launching stream; a loop's time is the maximum over the ranks, the
    # reported value is the median loop. NVML is sampled every 2 ms across all of them.
    repeats = args.repeats if args.repeats > 0 else 7
    if args.repeats <= 0:
        # short loops (small workloads): more of them, so that the loops together last ~40 ms and NVML gets its samples
        t0_, t1_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0_.record()
        for i in range(args.steps):
            run_step(i)
        t1_.record()
        torch.cuda.synchronize()
        est = max(t0_.elapsed_time(t1_) * 1e-3, 1e-6)
        repeats = int(wdist.max_over_ranks(float(max(7, min(200, int(0.04 / est) + 1))), dev))
    loop_sec = []
    with clocks:
        for _ in range(repeats):
            wdist.barrier(dev)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(args.steps):
                run_step(i)
            e1.record()
            torch.cuda.synchronize()
            wdist.barrier(dev)
            loop_sec.append(wdist.max_over_ranks(e0.elapsed_time(e1) * 1e-3, dev))
    sec = statistics.median(loop_sec)
    # the SM clock the GEMMs really ran at (cycle counter over nanosecond timer, stamped by the kernel itself)
    gemm_mhz = [c[0] for layer in sets for L in layer if L["spec"].M > 8 for c in [w8.gemm_clock_stamps(L["ws"])] if c]
    for layer in sets:
        for L in layer:
            st = w8.int8_check_status(L["ws"])
            if st != 0:
                raise SystemExit(f"device-side status: {w8.status_string(st)}")
    if w8.int8_sticky_status(clear=True) != 0:          # a time-out of ANY call of the loops, not only the last ones
        raise SystemExit("device-side status: a bounded wait expired during the timed loops")
    # ---- the same steps as direct calls, straight after (same thermal state): what a caller without graphs gets
    direct = None
    if graphs is not None and rank == 0:
        for i in range(5):
            step(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(args.steps):
            step(i)
        b.record()
        torch.cuda.synchronize()
        d_sec = a.elapsed_time(b) * 1e-3 / args.steps
        direct = {"value": ops_per_step / d_sec / 1e12, "unit": "TOPS", "ms_per_step": d_sec * 1e3, "steps": args.steps,
                  "note": "the step's int8_linear_fused calls issued one by one, timed right after the headline loop"}
    ops_all_ranks = wdist.sum_over_ranks(ops_per_step * args.steps, dev)
    tops = ops_all_ranks / sec / 1e12
    # quantizer + GEMM per linear; one launch where the shape takes the one-kernel path
    launches = args.steps * sum(1 if "one kernel" in w8.int8_linear_plan(s_.M, s_.N, s_.K, w8.ACT_BF16)["name"] else 2
                                for s_ in specs)

    line = {
        "metric": METRIC, "value": tops, "unit": "TOPS", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": sec / args.steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8", "data": "synthetic",
        "config": {"workload": workload_name(args.workload, specs), "entry": "int8_linear_fused from bf16 activations",
                   "launch": launch_note,
                   "regime": f"median of {repeats} back-to-back loops of --steps steps; a loop beyond ~200 steps (50 ms) runs "
                             "under the 1 kW power cap (see clocks)",
                   "l2": f"inputs larger than L2: {len(sets)} rotating sets of {set_bytes / 1e6:.0f} MB each",
                   "parallelism": f"dp{world} over tokens, weights replicated, no collective"},
        "pct_of_int8_peak": 100.0 * tops / (INT8_PEAK_TOPS * world), "int8_peak_tops": INT8_PEAK_TOPS,
        "clocks": clocks.summary(), "gpu_launches": launches, "gpu_launches_all_loops": launches * repeats,
        "repeats": {"loops": repeats, "ms_per_step": [t / args.steps * 1e3 for t in loop_sec],
                    "tops": [ops_all_ranks / t / 1e12 for t in loop_sec], "reported": "median"},
    }
    # What the tensor pipes could do at the clock seen: 16384 int8 ops per clock per SM (8192 multiply-adds). Two
    # clocks: NVML's (the PLL setting, sampled every 2 ms over the loops) and the one the GEMM kernels measured
    # themselves (cycles over nanoseconds inside the launch), which is lower under a dense tensor load.
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    if line["clocks"]["sm_mhz"]:
        ceiling = sms * 16384 * line["clocks"]["sm_mhz"] * 1e6 / 1e12
        line["int8_ceiling_at_observed_clock"] = {"tops": ceiling, "sm_mhz": line["clocks"]["sm_mhz"], "sms": sms,
                                                  "clock_source": "NVML, median of the samples taken during the timed loops",
                                                  "value_frac": tops / (ceiling * world)}
    if gemm_mhz:
        mhz = statistics.median(gemm_mhz)
        ceiling = sms * 16384 * mhz * 1e6 / 1e12
        line["int8_ceiling_at_kernel_clock"] = {"tops": ceiling, "sm_mhz": mhz, "sms": sms,
                                                "clock_source": "SM cycle counter / nanosecond timer inside the last GEMM launches of the timed loops",
                                                "value_frac": tops / (ceiling * world)}

    if burst is not None and rank == 0:
        line["burst"] = burst
    if direct is not None:
        line["direct_calls"] = direct
    if rank == 0:
        # ---- per-kernel timing (same kernels, same launch configuration, timed one by one)
        per_shape, gemm_ops, gemm_sec, q_bytes, q_sec = [], 0.0, 0.0, 0.0, 0.0
        for j, spec in enumerate(specs):
            M, K, N = spec.M, spec.K, spec.N
            s_off, q_off = w8.int8_linear_workspace_offsets(M, K)
            rot = [sets[r][j] for r in range(len(sets))]
            views = [(L, L["ws"][s_off:s_off + 4 * M].view(torch.float32), L["ws"][q_off:q_off + M * K].view(torch.int8).view(M, K))
                     for L in rot]
            ws8 = w8.alloc_workspace(M, N, K, w8.ACT_INT8, dev)
            it = [0]
            g_args = [fused_args(L, bf16=False, s_tok=st_, qa=qa_, ws=ws8) for (L, st_, qa_) in views]
            q_args = [(L["A"].data_ptr(), M, K, K, qa_.data_ptr(), st_.data_ptr(), stream) for (L, st_, qa_) in views]
            f_args = [fused_args(L) for (L, _, _) in views]
            # the one-pass quantizer takes the absmax of every row from the producer of the activations; here the set-up
            # computes it (exactly: bf16 widens to fp32 without rounding and a maximum does not round)
            rowmax = [L["A"].float().abs().amax(dim=1).contiguous() for (L, _, _) in views]
            q1_args = [(L["A"].data_ptr(), M, K, K, rm.data_ptr(), qa_.data_ptr(), st_.data_ptr(), stream)
                       for (L, st_, qa_), rm in zip(views, rowmax)]

            def gemm_only():
                it[0] += 1
                raw.int8_linear_fused(*g_args[it[0] % len(g_args)])

            def gemm_hot():                       # same buffers every time: operands stay in L2 where they fit
                raw.int8_linear_fused(*g_args[0])

            def quant_only():
                it[0] += 1
                raw.int8_quantize_act_per_token(*q_args[it[0] % len(q_args)])

            def quant_one_pass():
                it[0] += 1
                raw.int8_quantize_act_per_token_given_absmax(*q1_args[it[0] % len(q1_args)])

            def fused():
                it[0] += 1
                raw.int8_linear_fused(*f_args[it[0] % len(f_args)])

            # back-to-back launches between one pair of events: the mean includes launch gaps, as in a model
            def batch_time(fn, n=60, warm=10):
                for _ in range(warm):
                    fn()
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for _ in range(n):
                    fn()
                b.record()
                torch.cuda.synchronize()
                return a.elapsed_time(b) * 1e-3 / n

            tg = batch_time(gemm_only)
            stamp = w8.gemm_clock_stamps(ws8) if M > 8 else None
            # the same launches on operands that do not toggle (all codes 1): what the kernel does when the data costs
            # no power, i.e. how much of the time above is the clock the chip allows on real operands
            const_ops = None
            if not args.no_extras and M > 16:
                L0 = rot[0]
                ones_a = torch.ones((M, K), dtype=torch.int8, device=dev)
                ones_w = torch.ones((N, K), dtype=torch.int8, device=dev)
                c_args = (ones_a.data_ptr(), 1, K, views[0][1].data_ptr(), ones_w.data_ptr(), L0["s_ch"].data_ptr(),
                          None if L0["bias"] is None else L0["bias"].data_ptr(), L0["out"].data_ptr(), N, M, N, K,
                          ws8.data_ptr(), ws8.numel(), stream)
                tc_ = batch_time(lambda: raw.int8_linear_fused(*c_args))
                cst = w8.gemm_clock_stamps(ws8)
                const_ops = {"us": tc_ * 1e6, "tops": spec.ops / tc_ / 1e12, "gemm_sm_mhz": cst[0] if cst else None}
                del ones_a, ones_w
            tgh = batch_time(gemm_hot)
            tq = batch_time(quant_only)
            tq1 = batch_time(quant_one_pass)
            tf_ = batch_time(fused)
            plan = w8.int8_linear_plan(M, N, K, w8.ACT_BF16, rot[0]["ws"].numel())
            per_shape.append({"name": spec.name, "M": M, "K": K, "N": N,
                              "kernel_config": plan["name"], "cta_groups": plan["groups"],
                              "k_split": f"{plan['split_tiles']} tiles x {plan['split_parts']} parts" if plan["split_parts"] else "none",
                              "fused_from_bf16_us": tf_ * 1e6, "fused_from_bf16_tops": spec.ops / tf_ / 1e12,
                              "pct_of_int8_peak": 100.0 * spec.ops / tf_ / 1e12 / INT8_PEAK_TOPS,
                              "gemm_epilogue_us": tg * 1e6, "gemm_epilogue_tops": spec.ops / tg / 1e12,
                              "gemm_sm_mhz": stamp[0] if stamp else None,
                              "gemm_first_cta_us": stamp[1] * 1e6 if stamp else None,
                              "gemm_epilogue_hot_l2_us": tgh * 1e6, "gemm_epilogue_hot_l2_tops": spec.ops / tgh / 1e12,
                              "gemm_epilogue_constant_operands": const_ops,
                              "quantizer_us": tq * 1e6, "quantizer_gbs": model.quantizer_bytes(M, K) / tq / 1e9,
                              "quantizer_given_absmax_us": tq1 * 1e6,
                              "quantizer_given_absmax_gbs": (model.quantizer_bytes(M, K) + 4 * M) / tq1 / 1e9})
            if M > 16:
                gemm_ops += spec.ops
                gemm_sec += tg
            q_bytes += model.quantizer_bytes(M, K)
            q_sec += tq
        line["per_shape"] = per_shape
        # The per-shape GEMM timings above are bursts (60 back-to-back launches, a few milliseconds): they belong with
        # the burst bf16 rate. The nominal int8 : bf16 ratio of the tensor pipes is 2. The long-loop (power-capped)
        # peak and the datasheet figure are quoted beside it, each with the fraction it gives.
        peak_burst = 2.0 * peaks["bf16_tflops"]
        peak_sustained = 2.0 * peaks["bf16_tflops_sustained"]
        achieved = gemm_ops / gemm_sec / 1e12 if gemm_sec > 0 else 0.0
        traffic = NCU_GEMM_DRAM_TRAFFIC.get(args.workload) if args.rows == 0 else None
        line["roofline"] = {
            "kernel": "gemm_tc_kernel (tcgen05.mma.kind::i8 + dequant epilogue)", "bound": "tensor",
            "achieved": achieved, "peak": peak_burst, "unit": "TFLOP/s", "frac": achieved / peak_burst if peak_burst else None,
            "regime": "burst: per-shape loops of 60 back-to-back pre-quantized launches on rotating buffers, CUDA events "
                      "around each loop; achieved = sum of 2*M*N*K over the shapes / sum of their mean launch times",
            "peak_source": f"2 x {peaks['source']} burst bf16 cuBLAS rate ({peaks['bf16_tflops']} TFLOP/s), of {peaks['source']}; "
                           "int8 multiply-add counted as 2 ops",
            "ops_per_launch_sum": gemm_ops, "seconds_per_launch_sum": gemm_sec,
            "frac_of_sustained_peak": {"peak": peak_sustained, "frac": achieved / peak_sustained,
                                       "note": "2 x the seconds-long power-capped bf16 rate: the ceiling of a launch inside a long loop, "
                                               "not of this burst measurement"},
            "frac_of_datasheet": {"peak": INT8_PEAK_TOPS, "frac": achieved / INT8_PEAK_TOPS},
            "traffic": traffic["bytes_per_launch"] if traffic else None,
            "traffic_source": (f"{traffic['profile']}: {traffic['note']}" if traffic else
                               "no ncu capture of this workload: not quoted"),
            "quantizer": {"bound": "hbm", "achieved": q_bytes / q_sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                          "frac": q_bytes / q_sec / 1e9 / peaks["hbm_gbs"],
                          "regime": "burst: 60 back-to-back launches per shape on rotating inputs",
                          "bytes_per_launch_sum": q_bytes, "seconds_per_launch_sum": q_sec},
        }
        clk = [p_["gemm_sm_mhz"] for p_ in per_shape if p_.get("gemm_sm_mhz")]
        if clk:
            ceiling = sms * 16384 * statistics.median(clk) * 1e6 / 1e12
            line["roofline"]["frac_of_pipe_peak_at_kernel_clock"] = {
                "peak": ceiling, "sm_mhz": statistics.median(clk), "frac": achieved / ceiling,
                "note": "148 SMs x 16384 int8 ops per clock x the SM clock the GEMM launches measured themselves"}
        if health is not None:
            line["health"] = health

        if not args.no_extras:
            # ---- end to end through the host-buffer entry point: pinned host activations in, host result out
            # Two copies of every linear's buffers (host and device) where the run has two input sets: consecutive
            # steps then share nothing, and a step's uploads need not wait for the previous step's downloads.
            copies = min(2, len(sets))
            e2e_sets = []
            for c in range(copies):
                row = []
                for L in sets[c]:
                    spec = L["spec"]
                    row.append({"L": L, "A_host": L["A"].cpu().pin_memory(),
                                "out_host": torch.empty((spec.M, spec.N), dtype=torch.bfloat16).pin_memory(),
                                "d_A": torch.empty_like(L["A"])})
                e2e_sets.append(row)

            # the linears of a step go to two streams in turn (and the next step to two others), so that one linear's
            # download overlaps another one's upload (PCIe is full duplex); every call in flight has its own
            # workspace, device and host buffers
            main_stream = torch.cuda.current_stream(dev)
            side = [torch.cuda.Stream(dev) for _ in range(2 * copies)]
            e2e_calls = [0]

            def e2e_step():
                c = e2e_calls[0] % copies
                e2e_calls[0] += 1
                for i, e in enumerate(e2e_sets[c]):
                    L = e["L"]
                    with torch.cuda.stream(side[2 * c + i % 2]):
                        w8.int8_linear_fused_host(e["A_host"], e["d_A"], L["qw"], L["s_ch"], L["bias"], L["out"], e["out_host"], L["ws"])

            def fork():
                ev = torch.cuda.Event()
                ev.record(main_stream)
                for s_ in side:
                    s_.wait_event(ev)

            def join():
                for s_ in side:
                    ev = torch.cuda.Event()
                    ev.record(s_)
                    main_stream.wait_event(ev)

            n_e2e = 10
            fork()
            for _ in range(3):
                e2e_step()
            join()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.perf_counter()
            a.record(main_stream)
            fork()
            for _ in range(n_e2e):
                e2e_step()
            join()
            b.record(main_stream)
            torch.cuda.synchronize()
            wall = time.perf_counter() - t0
            e2e_sec = max(a.elapsed_time(b) * 1e-3, wall) / n_e2e
            line["e2e"] = {"value": ops_per_step / e2e_sec / 1e12, "unit": "TOPS",
                           "h2d_bytes_per_step": sum(2 * s.M * s.K for s in specs),
                           "d2h_bytes_per_step": sum(2 * s.M * s.N for s in specs), "ms_per_step": e2e_sec * 1e3,
                           "entry": "int8_linear_fused_host (pinned host bf16 in, pinned host bf16 out), linears alternating over "
                                    f"{len(side)} streams, {copies} sets of buffers"}

            # ---- context on the same box: library bf16 matmul and library int8 matmul on the same shapes
            ctx = []
            for L in sets[0]:
                spec = L["spec"]
                if spec.M <= 16:
                    continue
                Wb = torch.randn(spec.N, spec.K, device=dev, dtype=torch.bfloat16)
                tb = statistics.mean(cuda_timer(torch, lambda: torch.matmul(L["A"], Wb.t()), 10, 3))
                s_off, q_off = w8.int8_linear_workspace_offsets(spec.M, spec.K)
                qa = L["ws"][q_off:q_off + spec.M * spec.K].view(torch.int8).view(spec.M, spec.K)
                ti = statistics.mean(cuda_timer(torch, lambda: torch._int_mm(qa, L["qw"].t()), 10, 3))
                # the unfused route the paper compares with: library integer matmul, then a separate dequantization pass
                s_tok_v = L["ws"][s_off:s_off + 4 * spec.M].view(torch.float32)

                def unfused():
                    acc = torch._int_mm(qa, L["qw"].t())
                    y = acc.float() * s_tok_v[:, None] * L["s_ch"][None, :]
                    if L["bias"] is not None:
                        y = y + L["bias"][None, :]
                    return y.to(torch.bfloat16)

                tu = statistics.mean(cuda_timer(torch, unfused, 6, 2))
                mine = next(p for p in per_shape if p["name"] == spec.name)
                ctx.append({"name": spec.name, "torch_bf16_matmul_tflops": spec.ops / tb / 1e12,
                            "torch_int_mm_tops_no_dequant": spec.ops / ti / 1e12,
                            "unfused_int_mm_plus_dequant_us": tu * 1e6,
                            "gemm_epilogue_speedup_over_unfused": tu / (mine["gemm_epilogue_us"] * 1e-6),
                            # the paper's Table 1 quantity on this machine: fused int8 linear over library bf16 matmul
                            "fused_from_bf16_speedup_over_bf16_matmul": tb / (mine["fused_from_bf16_us"] * 1e-6),
                            "gemm_epilogue_speedup_over_bf16_matmul": tb / (mine["gemm_epilogue_us"] * 1e-6)})
                del Wb
            line["context"] = ctx

            # ---- the oracle on the host cores, bounded sample (only at one GPU)
            if world == 1:
                v, sec_o, cores, sample = time_oracle(specs, 1, 0, target_gmac=400.0)
                line["cpu_baseline"] = {"value": v, "unit": "TOPS", "cores": cores, "kind": "oracle", "sample": sample,
                                        "seconds": sec_o}
        print(json.dumps(line), flush=True)
    wdist.barrier(dev)


if __name__ == "__main__":
    main()
