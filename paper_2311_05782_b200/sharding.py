"""Trial sharding across ranks (one process per GPU) and the cross-rank reductions of the benchmark.

Trials are independent (one fault per trial), so a campaign shards by contiguous ranges of the
trial table with the operands replicated; no collective is needed on the data path. The only
cross-rank exchanges are the max of the elapsed time and the sum of the work done.
"""
from __future__ import annotations


def shard_range(n_items: int, rank: int, world: int):
    """Contiguous [lo, hi) share of n_items for `rank`; sizes differ by at most one."""
    if world <= 0 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    base, extra = divmod(n_items, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def _reduce(value: float, world: int, device, op_name: str) -> float:
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=getattr(dist.ReduceOp, op_name))
    return float(t.item())


def reduce_max(value: float, world: int, device="cpu") -> float:
    """Max over ranks (the job is as slow as its slowest rank)."""
    return _reduce(value, world, device, "MAX")


def reduce_sum(value: float, world: int, device="cpu") -> float:
    """Sum over ranks (whole-job units of work)."""
    return _reduce(value, world, device, "SUM")


def gather_records(local_records, world: int):
    """Concatenate per-rank trial records (numpy structured arrays) in rank order on every rank."""
    if world <= 1:
        return local_records
    import numpy as np
    import torch.distributed as dist
    parts = [None] * world
    dist.all_gather_object(parts, local_records)
    return np.concatenate(parts)
