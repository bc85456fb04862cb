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


def init(backend: str):
    """Joins the process group described by RANK / WORLD_SIZE / MASTER_* when there is more than one rank."""
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        kw = {}
        if backend == "nccl":
            kw["device_id"] = torch.device("cuda", local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)
    return rank, local_rank, world


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
