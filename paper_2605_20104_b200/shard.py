"""Host-side sharding of the verify path over ranks (one process per GPU).

Sequences are independent within a step (only the adjacency matrix is shared, and it is read-only
inside a step, so it is replicated): ranks never exchange data on the path.  torch.distributed is
used for two things only: a barrier around the timed region and the max over ranks of a device
time.  These helpers hold that logic so that it can be exercised with gloo on CPU.
"""
from __future__ import annotations

from typing import List, Tuple

import torch


def rank_seed(base_seed: int, rank: int) -> int:
    """Weak scaling: every rank verifies its own batch of the same shape, drawn from its own seed."""
    return base_seed + 1009 * rank


def split_batch(B: int, world: int) -> List[Tuple[int, int]]:
    """Strong scaling: contiguous [lo, hi) sequence ranges, sizes differing by at most one."""
    base, extra = divmod(B, world)
    out, lo = [], 0
    for r in range(world):
        hi = lo + base + (1 if r < extra else 0)
        out.append((lo, hi))
        lo = hi
    return out


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """Max of a per-rank scalar (the device time of the timed region) over the default group."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: str = "cpu") -> float:
    """Sum of a per-rank scalar (units processed) over the default group."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
