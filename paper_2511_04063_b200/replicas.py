"""Host-side logic of multi-GPU runs.  The calibration path has no exchange step between
GPUs: every rank calibrates its own rotation site (an independent seeded problem), so N GPUs
are N replicas and the only collective is the max over ranks of the measured times."""
from __future__ import annotations

from dataclasses import replace


def workload_for_rank(w, rank: int):
    """The problem rank `rank` calibrates: same recipe, its own seed (rank 0 keeps the base seed)."""
    return replace(w, seed=w.seed + rank)


def max_over_ranks(values, device="cpu"):
    """Element-wise max of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_rate(units_per_rank: float, world: int, ms_max: float) -> float:
    """Units all ranks processed divided by the slowest rank's time (weak scaling)."""
    return world * units_per_rank / (ms_max * 1e-3)
