"""The N > 1 host path on gloo ranks: trial sharding, the sharded campaign's record gather (one all_gather of padded
byte blocks), max-over-ranks time and summed work. The library's campaign call is replaced by a callable that needs no
GPU (it fills the records from the oracle), so what runs here is the product's own host code."""
import os
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

from paper_2311_05782_b200.sharding import shard_range


def test_shard_range_partitions_exactly():
    for n in (0, 1, 7, 1024, 100000):
        for world in (1, 2, 3, 8):
            spans = [shard_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[r][1] == spans[r + 1][0] for r in range(world - 1))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_range(10, 3, 3)


def _worker(rank, world, port, out, n_trials):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import oracle as orc
    import synth
    from paper_2311_05782_b200.sharding import campaign_sharded, reduce_max, reduce_sum, shard_range
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.make_workload("c5", 96, 64, 64, trials=max(n_trials, 1))
    sites = w.sites[:n_trials]
    Cc, *_ = orc.gemm(w.dtype, w.A, w.Bt)
    calls = []

    def run_local(dtype, A, Bt, share, mode):
        # stands in for mpgemmfi_campaign: same contract (clean product, int32 [n, 12] records of the share)
        n = 0 if share is None else len(share)
        calls.append(n)
        rec = orc.campaign(dtype, A, Bt, Cc, share, mode) if n else np.zeros(0, dtype=orc.RECORD)
        return torch.from_numpy(Cc), torch.from_numpy(rec.view(np.int32).reshape(n, 12).copy())

    _, allrec = campaign_sharded(w.dtype, w.A, w.Bt, sites if n_trials else None, w.detect_mode, run_local=run_local)
    lo, hi = shard_range(n_trials, rank, world)
    t = reduce_max(10.0 + rank, world)
    units = reduce_sum(float(hi - lo), world)
    full = orc.campaign(w.dtype, w.A, w.Bt, Cc, sites, w.detect_mode) if n_trials else np.zeros(0, dtype=orc.RECORD)
    ok = (np.array_equal(allrec.numpy().view(np.uint8).reshape(-1), full.view(np.uint8).reshape(-1))
          and tuple(allrec.shape) == (n_trials, 12) and calls == [hi - lo]
          and t == 10.0 + world - 1 and units == float(n_trials))
    with open(f"{out}.{rank}", "w") as f:
        f.write("ok" if ok else f"bad {t} {units} {tuple(allrec.shape)} {calls}")
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,n_trials", [(2, 33), (3, 100), (3, 2), (2, 0), (2, 64)])
def test_sharded_campaign_reassembles_the_records(tmp_path, world, n_trials):
    """Even and uneven splits, ranks with no trials at all, an empty table: every rank ends with the records of the
    whole table, in table order, equal to an unsharded run."""
    out = str(tmp_path / "result")
    port = 29500 + (os.getpid() * 7 + world * 131 + n_trials) % 2000
    mp.spawn(_worker, args=(world, port, out, n_trials), nprocs=world, join=True)
    for r in range(world):
        assert open(f"{out}.{r}").read() == "ok", r
