"""The N > 1 host path (trial sharding, max-over-ranks time, summed work, record gather) on two gloo ranks."""
import os
import sys

import numpy as np
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


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import oracle as orc
    import synth
    from paper_2311_05782_b200.sharding import gather_records, reduce_max, reduce_sum, shard_range
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.make_workload("c1", 64, 64, 64, trials=33)
    lo, hi = shard_range(len(w.sites), rank, world)
    Cc, *_ = orc.gemm(w.dtype, w.A, w.Bt)
    rec = orc.campaign(w.dtype, w.A, w.Bt, Cc, w.sites[lo:hi], w.detect_mode)      # this rank's trials
    allrec = gather_records(rec, world)
    t = reduce_max(10.0 + rank, world)
    units = reduce_sum(float(hi - lo), world)
    if rank == 0:
        full = orc.campaign(w.dtype, w.A, w.Bt, Cc, w.sites, w.detect_mode)
        ok = np.array_equal(allrec.view(np.uint8), full.view(np.uint8)) and t == 10.0 + world - 1 and units == 33.0
        with open(out, "w") as f:
            f.write("ok" if ok else f"bad {t} {units} {len(allrec)}")
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_campaign_shards_reassemble(tmp_path):
    out = str(tmp_path / "result.txt")
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert open(out).read() == "ok"
