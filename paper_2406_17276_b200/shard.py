"""Host-side logic of a multi-process run: one process per GPU, every process builds trees for
its own sequences.  Sequences never exchange data (Algorithm 1 works on one sequence), so there
is no collective on the data path; the processes only meet to time the job: a barrier on both
sides of the timed region, the slowest rank's time, and the number of trees all ranks built.
"""
from __future__ import annotations

from .synth import Workload


def rank_workload(w: Workload, rank: int) -> Workload:
    """The workload of one rank: same shape, its own seed (its own tables and root tokens)."""
    return Workload(**{**w.__dict__, "seed": w.seed + 1000 * rank})


def max_over_ranks(x: float, device: str = "cpu") -> float:
    """The largest x of all ranks (x itself without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, device: str = "cpu") -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job(units_local: float, ms_local: float, device: str = "cpu") -> tuple[float, float]:
    """(units of all ranks per second, the slowest rank's milliseconds)."""
    ms = max_over_ranks(ms_local, device)
    units = sum_over_ranks(units_local, device)
    return units / (ms * 1e-3), ms
