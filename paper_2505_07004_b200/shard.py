"""Multi-GPU plumbing: the path shards over independent layers, one per rank, with no data-path
collective (the paper computes Hessians of different layers / groups on different GPUs, Section 3.2 and
Appendix C).  The only communication is the reduction of timings and of per-rank scalar results."""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def layer_seed_for_rank(base_seed: int, rank: int) -> int:
    """Every rank works on its own synthetic layer: distinct seeds, same shape."""
    return int(base_seed) + int(rank)


def max_over_ranks(values: Sequence[float], device="cpu") -> list:
    """Element-wise maximum over all ranks of a few host scalars (timings)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def gather_scalars(value: float, device="cpu") -> list:
    """All ranks' values of one host scalar, in rank order (e.g. each layer's objective)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(value)]
    t = torch.tensor([value], dtype=torch.float64, device=device)
    out = [torch.zeros_like(t) for _ in range(dist.get_world_size())]
    dist.all_gather(out, t)
    return [float(o.item()) for o in out]


def whole_job_throughput(units_per_rank: int, steps: int, max_seconds: float, world: int) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return float(units_per_rank) * world * steps / max_seconds
