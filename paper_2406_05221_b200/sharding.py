"""Host-side sharding of a workload over ranks (one process per GPU).

Tasksets are independent, so the analysis has no exchange step: every rank analyses its own
contiguous range of taskset indices and the only cross-rank traffic is the reduction of a few
scalars (elapsed time: max; counts: sum) through ``torch.distributed``.
"""
from __future__ import annotations

from typing import Sequence, Tuple


def weak_shard(rank: int, per_rank: int) -> Tuple[int, int]:
    """(first, count) of rank ``rank`` when every rank analyses ``per_rank`` tasksets of the same
    generator stream (weak scaling: the job grows with the number of ranks)."""
    if rank < 0 or per_rank < 0:
        raise ValueError("rank and per_rank must be non-negative")
    return rank * per_rank, per_rank


def strong_shard(rank: int, world: int, total: int) -> Tuple[int, int]:
    """(first, count) of rank ``rank`` when ``total`` tasksets are split as evenly as possible
    into ``world`` contiguous ranges (the first ``total % world`` ranks take one more)."""
    if not (0 <= rank < world) or total < 0:
        raise ValueError("bad rank/world/total")
    base, extra = divmod(total, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def reduce_scalars(values: Sequence[float], op: str, device=None):
    """All-reduces a short list of Python numbers over the default process group (``op`` is
    'max' or 'sum'); a no-op without an initialised group.  Returns a list of floats."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return [float(v) for v in t.cpu().tolist()]
