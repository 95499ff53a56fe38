"""Host-side helpers for running the path as independent replicas, one process per GPU.

The path has no exchange step, so ranks never communicate on the data path; these helpers
only aggregate timings (max over ranks) and assign streams to ranks."""
from __future__ import annotations

from typing import List, Sequence


def assign_streams(pair_counts: Sequence[int], world: int) -> List[List[int]]:
    """Greedy longest-first assignment of streams to ranks, balanced by causal-pair count
    (the work of a stream), not by token count.  Returns stream indices per rank."""
    order = sorted(range(len(pair_counts)), key=lambda i: (-pair_counts[i], i))
    load = [0] * world
    out: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda j: (load[j], j))
        out[r].append(i)
        load[r] += pair_counts[i]
    return [sorted(x) for x in out]


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Max of a per-rank scalar (device time of the timed region)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, seconds: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return units_per_rank * world / seconds
