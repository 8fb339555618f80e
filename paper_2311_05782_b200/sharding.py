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
    if dist.get_backend() != "nccl":
        device = "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=getattr(dist.ReduceOp, op_name))
    return float(t.item())


def reduce_max(value: float, world: int, device="cpu") -> float:
    """Max over ranks (the job is as slow as its slowest rank)."""
    return _reduce(value, world, device, "MAX")


def reduce_sum(value: float, world: int, device="cpu") -> float:
    """Sum over ranks (whole-job units of work)."""
    return _reduce(value, world, device, "SUM")


RECORD_BYTES = 48


def gather_records(local, counts, group=None):
    """All ranks' trial records in rank order, on every rank: ONE all_gather of fixed-size byte blocks.

    local: this rank's records as a uint8 tensor [n_local * 48] (or any tensor of that many bytes) on the device the
    process group communicates on (CUDA for nccl, CPU for gloo); counts: trials per rank (known to every rank from
    shard_range, so no size exchange is needed). Every rank contributes a block padded to the largest share; the
    padding is cut out after the gather. Returns a uint8 tensor [sum(counts) * 48]."""
    import torch
    import torch.distributed as dist
    world = len(counts)
    flat = local.reshape(-1).view(torch.uint8)
    if world <= 1:
        return flat
    block = max(counts) * RECORD_BYTES
    # the collective runs where the group's backend works: device memory for nccl, host memory for gloo (the records
    # then travel through the host and come back to the device they were on)
    home = flat.device
    coll = home if dist.get_backend(group) == "nccl" else torch.device("cpu")
    send = torch.zeros(block, dtype=torch.uint8, device=coll)
    send[:flat.numel()] = flat.to(coll)
    recv = torch.empty(world * block, dtype=torch.uint8, device=coll)
    dist.all_gather_into_tensor(recv, send, group=group)
    if not all(c == counts[0] for c in counts):
        recv = torch.cat([recv[r * block:r * block + counts[r] * RECORD_BYTES] for r in range(world)])
    return recv.to(home)


def campaign_sharded(dtype, A, Bt, sites, detect_mode, group=None, run_local=None):
    """A campaign whose trial table is shared out over the ranks of a process group (one process per GPU).

    Every rank holds the whole operands and the whole table (a numpy structured array of 32-byte sites), runs the clean
    GEMM and ITS contiguous share of the trials through mpgemmfi_campaign, and receives every rank's records through
    one all_gather. There is no other exchange: trials are independent. Returns (C_clean, records) with records an
    int32 tensor [n_trials, 12] in table order, identical on every rank.

    run_local(dtype, A, Bt, sites_share, detect_mode) -> (C_clean, records int32 [n, 12]) stands in for the library
    call in tests that have no GPU; the default is the library's campaign()."""
    import torch
    import torch.distributed as dist
    if run_local is None:
        from .binding import campaign as run_local
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    rank = dist.get_rank(group) if world > 1 else 0
    n = 0 if sites is None else len(sites)
    spans = [shard_range(n, r, world) for r in range(world)]
    lo, hi = spans[rank]
    C_clean, rec = run_local(dtype, A, Bt, sites[lo:hi] if n else None, detect_mode)
    rec = rec.reshape(-1, 12)[:hi - lo].contiguous()
    allrec = gather_records(rec, [b - a for a, b in spans], group)
    return C_clean, allrec.view(torch.int32).reshape(n, 12)
