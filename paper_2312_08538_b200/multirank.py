"""Rank plumbing.

``aggregate`` / ``throughput`` serve the benchmark, whose ranks run replicas of the workload (N
workers simulated on each device, no exchange): ranks only agree on the timing, the job's time is
the slowest rank's and its work the sum over ranks.  ``ShardedConEF`` is the other arrangement, one
worker per rank with the messages all-reduced across ranks."""
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


class WallClock:
    """Host clock for runs without a GPU."""

    def start(self):
        import time
        self.t0 = time.perf_counter()

    def stop_ms(self) -> float:
        import time
        return (time.perf_counter() - self.t0) * 1e3


class CudaClock:
    """CUDA events on the current stream of `device`, with a device synchronize on both sides."""

    def __init__(self, device):
        self.device = device

    def start(self):
        torch.cuda.synchronize(self.device)
        self.e0 = torch.cuda.Event(enable_timing=True)
        self.e1 = torch.cuda.Event(enable_timing=True)
        self.e0.record(torch.cuda.current_stream(self.device))

    def stop_ms(self) -> float:
        self.e1.record(torch.cuda.current_stream(self.device))
        torch.cuda.synchronize(self.device)
        return self.e0.elapsed_time(self.e1)


def timed_steps(step_fn, steps: int, warmup: int, clock, barrier=None) -> float:
    """Milliseconds per step of `step_fn(t)` over `steps` steps after `warmup`, bracketed by `barrier`
    (all ranks) and the clock's own synchronisation on both sides."""
    t = 0
    for _ in range(warmup):
        step_fn(t)
        t += 1
    if barrier is not None:
        barrier()
    clock.start()
    for _ in range(steps):
        step_fn(t)
        t += 1
    ms = clock.stop_ms()
    if barrier is not None:
        barrier()
    return ms / max(1, steps)


# ------------------------------------------------------------------ one worker per rank
MSG_VALUES, MSG_P, MSG_Q, MSG_DENSE1D = 0, 1, 2, 3


class ShardedConEF:
    """One ConEF worker per process; Alg. 2 line 7's Aggregate is an all-reduce over the ranks.

    ``engine`` is a context with ONE local worker (``binding.ConEF(..., n_workers=1)`` on a GPU; any
    object with the same methods elsewhere).  Every message of the local worker is summed over the
    ranks in place before the engine's own reduction call consumes it, and the engine is told the
    job's number of workers so that its means divide by it:

        random-k / identity:  step -> all-reduce(values, dense1d) -> reduce -> [apply_update]
        low-rank:             step(0) -> all-reduce(P_i) -> reduce(P) [Gram-Schmidt of the global sum]
                              -> step(1) -> all-reduce(Q_i) -> reduce(Q) [Q_t = sum / N] -> ...

    Only the small messages cross the network (k values, or (rows + cols) r factors per tensor); the
    compressed error never leaves its GPU.  The sum over ranks is the collective's, so results match
    a single-process run with N simulated workers up to the order of the fp32 additions.
    """

    def __init__(self, engine, lowrank: bool, world_size: int = None, all_reduce=None):
        self.eng = engine
        self.lowrank = bool(lowrank)
        if all_reduce is None:
            def all_reduce(t):
                dist.all_reduce(t, op=dist.ReduceOp.SUM)
        self.all_reduce = all_reduce
        if world_size is None:
            world_size = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
        self.world = int(world_size)
        self.eng.set_total_workers(self.world)

    def _sum_over_ranks(self, kind):
        if self.eng.message_elems(kind) > 0:
            self.all_reduce(self.eng.message(kind, 0))

    def step(self, t, grad, x=None):
        """One step of Alg. 2 for this rank's worker; returns {kind: summed message}.  With ``x``
        (this rank's copy of the flat parameters) the update x <- x - Delta_t is applied too."""
        out = {}
        self.eng.step(t, [grad], 0)
        self._sum_over_ranks(MSG_DENSE1D)
        if self.lowrank:
            self._sum_over_ranks(MSG_P)
            out[MSG_P] = self.eng.reduce_messages(MSG_P)
            self.eng.step(t, [grad], 1)
            self._sum_over_ranks(MSG_Q)
            out[MSG_Q] = self.eng.reduce_messages(MSG_Q)
        else:
            self._sum_over_ranks(MSG_VALUES)
            out[MSG_VALUES] = self.eng.reduce_messages(MSG_VALUES)
        if self.eng.message_elems(MSG_DENSE1D) > 0:
            out[MSG_DENSE1D] = self.eng.reduce_messages(MSG_DENSE1D)
        if x is not None:
            self.eng.apply_update(x, out)
        return out
