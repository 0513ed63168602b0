"""Host-side logic of a multi-GPU run: the path has no exchange step, so N GPUs are N replicas.

Every rank runs a full batch of its own seed; the only thing reduced across ranks is the timing
(max over ranks, so the job is as slow as its slowest replica).  No arithmetic of the method lives here.
"""
from __future__ import annotations

from . import workloads as wl

SEED_STRIDE = 1000


def rank_workload(w: wl.Workload, rank: int) -> wl.Workload:
    """The batch rank `rank` runs: same shapes, its own seed (rank 0 keeps the workload's seed)."""
    return w.replace(seed=w.seed + SEED_STRIDE * rank) if rank else w


def max_over_ranks(seconds: float, dist=None, device="cpu") -> float:
    """Slowest rank's time; `dist` is an initialised torch.distributed module or None (single process)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(seconds)
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def count_ranks(dist=None, device="cpu") -> int:
    """How many ranks really took part (each contributes one to a sum over the process group)."""
    if dist is None or not dist.is_initialized():
        return 1
    import torch
    t = torch.ones(1, dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())


def job_throughput(units_per_rank: int, world: int, seconds: float) -> float:
    """Whole-job units per second under weak scaling: every rank processed `units_per_rank` in `seconds`."""
    return world * units_per_rank / seconds
