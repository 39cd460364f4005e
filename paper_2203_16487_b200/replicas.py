"""Replica logic for more than one GPU: sequences never interact, so ranks decode disjoint
slices of the step stream and only timing and token counts are reduced (no data-path collective)."""
from __future__ import annotations

from typing import Tuple


def batch_index(step: int, rank: int, world: int, n_batches: int) -> int:
    """Batch that `rank` decodes at its `step`: the stream is dealt round-robin over the ranks."""
    return (step * world + rank) % max(n_batches, 1)


def reduce_job(tokens: float, ms: float, device=None) -> Tuple[float, float]:
    """(sum of tokens over ranks, max of elapsed ms over ranks); identity without a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(tokens), float(ms)
    t = torch.tensor([float(tokens)], dtype=torch.float64, device=device)
    m = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    dist.all_reduce(m, op=dist.ReduceOp.MAX)
    return float(t.item()), float(m.item())
