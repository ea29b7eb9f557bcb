"""Multi-GPU plumbing: the DES-LOC step shards by parameter range with no exchange step.

Every coordinate's update -- the average over the M replicas included -- touches only that
coordinate, so ranks can own disjoint slices of the tensor list (all M replicas of a slice on
one GPU) and step them independently; no data-path collective exists.  torch.distributed is
used only to agree on the slices and to reduce timings.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist

Slice = Tuple[int, int, int]  # (tensor index, first element, element count)


def shard_tensor_list(numel: Sequence[int], rank: int, world: int, align: int = 4096) -> List[Slice]:
    """Rank `rank`'s slices when the flat parameter range is cut into `world` near-equal parts.

    Cuts fall on multiples of `align` elements within a tensor (or on tensor ends), so every
    slice keeps 16-byte alignment and whole chunks.  The union over ranks covers every element
    exactly once; a rank may get nothing when there are fewer aligned units than ranks.
    """
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    total_units = sum(-(-int(n) // align) for n in numel)
    lo = total_units * rank // world
    hi = total_units * (rank + 1) // world
    out: List[Slice] = []
    pos = 0
    for k, n in enumerate(numel):
        nu = -(-int(n) // align)
        a, b = max(lo, pos), min(hi, pos + nu)
        if a < b:
            start = (a - pos) * align
            end = min(int(n), (b - pos) * align)
            out.append((k, start, end - start))
        pos += nu
    return out


def max_over_ranks(value: float, device=None) -> float:
    """max over ranks of a timing (every multi-GPU number is the slowest rank's)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: int, device=None) -> int:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return int(value)
    t = torch.tensor([value], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())


def whole_job_rate(units_per_rank: int, steps: int, local_ms: float, device=None) -> float:
    """Units per second of the whole job: all ranks' units over the slowest rank's time."""
    ms = max_over_ranks(local_ms, device)
    units = sum_over_ranks(units_per_rank, device)
    return units * steps / (ms * 1e-3)
