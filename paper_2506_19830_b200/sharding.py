"""How the verify pass spreads over several GPUs: by request, with no exchange on the data path.

Requests do not interact in any of the three steps, so every rank (one process per GPU) owns whole
requests and runs the same three calls on them.  The only traffic between ranks is the reduction
of the measurements: the step time of the job is the slowest rank's, its throughput the sum of
the ranks' verified tokens over that time.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the independent synthetic batch of ``rank`` (weak scaling: one batch per rank)."""
    return int(base_seed) + 1000 * int(rank)


def shard_requests(n_requests: int, world: int) -> List[Tuple[int, int]]:
    """Contiguous, balanced request ranges ``[begin, end)`` for ranks 0..world-1 (sizes differ by at most 1)."""
    if world < 1 or n_requests < 0:
        raise ValueError("world must be >= 1 and n_requests >= 0")
    base, extra = divmod(n_requests, world)
    out, begin = [], 0
    for r in range(world):
        n = base + (1 if r < extra else 0)
        out.append((begin, begin + n))
        begin += n
    return out


def reduce_measurement(ms_local: float, units_local: float, device="cpu") -> Tuple[float, float]:
    """(max over ranks of ms_local, sum over ranks of units_local).  Without an initialised process
    group the local values are returned."""
    t = torch.tensor([float(ms_local)], device=device, dtype=torch.float64)
    u = torch.tensor([float(units_local)], device=device, dtype=torch.float64)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def job_throughput(ms_per_step_max: float, units_total: float) -> float:
    """Whole-job units per second from the slowest rank's step time."""
    return units_total / (ms_per_step_max * 1e-3)
