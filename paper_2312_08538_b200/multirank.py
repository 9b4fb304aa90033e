"""Rank plumbing of the benchmark when several GPUs run replicas of the workload.

The ConEF step built here has no cross-GPU exchange (N workers are simulated on
one device), so ranks only agree on the timing: the job's time is the slowest
rank's, its work is the sum over ranks."""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def aggregate(ms: float, units: float, device="cpu") -> Tuple[float, float]:
    """(max over ranks of ms, sum over ranks of units); identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms), float(units)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def throughput(ms_per_step: float, units_per_step_per_rank: float, device="cpu") -> Tuple[float, float]:
    """Whole-job units per second and the step time it is based on."""
    ms, units = aggregate(ms_per_step, units_per_step_per_rank, device)
    return units / (ms * 1e-3), ms
