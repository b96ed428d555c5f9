"""Host-side helpers for running one independent verification batch per GPU.

The path has no exchange step (requests are independent; the paper moves state
between workers through the host, not between GPUs), so ranks share nothing on
the data path.  torch.distributed is used only to line the ranks up and to
combine their timings: the job's time is the slowest rank's, its work is the
sum.  Works on any backend (nccl on GPUs, gloo on CPU in the tests)."""
from __future__ import annotations

from dataclasses import replace
from typing import Tuple


def rank_seed(base_seed: int, rank: int) -> int:
    """Each rank draws its own batch: same shape and distributions, different seed."""
    return base_seed + 1000 * rank


def rank_config(cfg, rank: int):
    return cfg if rank == 0 else replace(cfg, seed=rank_seed(cfg.seed, rank))


def combine(ms_local: float, units_local: float, device=None) -> Tuple[float, float]:
    """(max over ranks of ms_local, sum over ranks of units_local); identity without a process group."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), float(units_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def job_throughput(ms_local: float, units_local: float, device=None) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    ms, units = combine(ms_local, units_local, device)
    return units / (ms * 1e-3)
