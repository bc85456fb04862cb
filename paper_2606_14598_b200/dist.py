"""Multi-GPU plumbing for the benchmark: one process per GPU, no data-path collective.

The fused linear is row-local (per-token scales, GEMM rows and epilogue rows never mix), so the path
shards over tokens: every rank runs the same kernels on its own rows with replicated weights. The
only communication is the benchmark's own barrier and reductions of scalars.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the launcher's environment (defaults: single process)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


RDZV_FILE_ENV = "W8A8_RDZV_FILE"


def init(backend: str):
    """Joins the process group described by RANK / WORLD_SIZE when there is more than one rank. The ranks meet
    through MASTER_ADDR / MASTER_PORT (a launcher such as torchrun sets them), or, when W8A8_RDZV_FILE names a
    fresh file, through that file: no port has to be picked ahead of time, so nothing can take it first."""
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        kw = {}
        if backend == "nccl":
            kw["device_id"] = torch.device("cuda", local_rank)
        rdzv = os.environ.get(RDZV_FILE_ENV)
        if rdzv:
            kw["init_method"] = "file://" + rdzv
        else:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return rank, local_rank, world


def spawn_ranks(argv, world: int, extra_env: dict | None = None, timeout: float | None = None):
    """Runs `argv` as `world` processes, one per rank (rank i is meant for GPU i), that meet through a rendezvous
    file. Returns [(returncode, stdout, stderr)] by rank. The children of a failed job are not left behind."""
    import subprocess
    import tempfile
    with tempfile.TemporaryDirectory(prefix="w8a8_rdzv_") as d:
        procs = []
        for r in range(world):
            env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world))
            env[RDZV_FILE_ENV] = os.path.join(d, "store")
            for k in ("MASTER_ADDR", "MASTER_PORT"):
                env.pop(k, None)
            env.update(extra_env or {})
            procs.append(subprocess.Popen(argv, env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
        out = []
        try:
            for p in procs:
                o, e = p.communicate(timeout=timeout)
                out.append((p.returncode, o, e))
        finally:
            for p in procs:
                if p.poll() is None:
                    p.kill()
                    p.wait()
        return out


def shard_rows(M: int, rank: int, world: int, multiple: int = 1):
    """Contiguous row range [lo, hi) of rank `rank` when M tokens are split over `world` ranks.
    Ranges are balanced to within `multiple` rows, cover [0, M) exactly and do not overlap."""
    units = (M + multiple - 1) // multiple
    base, extra = divmod(units, world)
    lo_u = rank * base + min(rank, extra)
    hi_u = lo_u + base + (1 if rank < extra else 0)
    return min(lo_u * multiple, M), min(hi_u * multiple, M)


def barrier(device=None):
    if dist.is_initialized():
        if device is not None and torch.device(device).type == "cuda":
            dist.barrier(device_ids=[torch.device(device).index])
        else:
            dist.barrier()


def _reduce(x: float, op, device):
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(x: float, device="cpu") -> float:
    return _reduce(x, dist.ReduceOp.MAX, device)


def sum_over_ranks(x: float, device="cpu") -> float:
    return _reduce(x, dist.ReduceOp.SUM, device)


def aggregate_throughput(units_this_rank: float, seconds_this_rank: float, device="cpu") -> tuple[float, float]:
    """Whole-job throughput: units of all ranks divided by the slowest rank's time. Returns (value, max seconds)."""
    total = sum_over_ranks(units_this_rank, device)
    t = max_over_ranks(seconds_this_rank, device)
    return total / t, t
