"""The N > 1 path on CPU: two gloo ranks shard a workload, analyse their shards independently
(with the CPU oracle standing in for the GPU library, which cannot run here) and reduce a few
scalars.  The union of the shards must equal the single-process result."""
import os
import socket
import sys

import numpy as np
import pytest

from paper_2406_05221_b200 import sharding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_arithmetic():
    assert sharding.weak_shard(0, 1000) == (0, 1000)
    assert sharding.weak_shard(3, 1000) == (3000, 1000)
    covered = []
    for world in (1, 2, 3, 8):
        for total in (0, 1, 7, 8, 1000, 1001):
            parts = [sharding.strong_shard(r, world, total) for r in range(world)]
            assert sum(c for _, c in parts) == total
            nxt = 0
            for first, count in parts:
                assert first == nxt
                nxt += count
            sizes = [c for _, c in parts]
            assert max(sizes) - min(sizes) <= 1
            covered.append(total)
    with pytest.raises(ValueError):
        sharding.strong_shard(2, 2, 10)
    assert sharding.reduce_scalars([1.5, 2.0], "max") == [1.5, 2.0]   # no process group: identity


def _worker(rank, world, port, per_rank, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from oracle import rta
    from paper_2406_05221_b200 import sharding, taskgen
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    w = taskgen.WORKLOADS["sweep"]
    first, count = sharding.weak_shard(rank, per_rank)
    batch = w.generate(first, count, stream=1)
    wcrt, sched, _ = rta.analyse(batch, rta.POLICY_GCAPS, w.timeslice_us, w.overhead_us)
    n_sched = float((sched == 1).sum())
    total_sched, total_sets = sharding.reduce_scalars([n_sched, float(count)], "sum")
    slowest = sharding.reduce_scalars([float(rank + 1)], "max")[0]
    np.save(os.path.join(out_dir, "wcrt_%d.npy" % rank), wcrt)
    if rank == 0:
        np.save(os.path.join(out_dir, "totals.npy"), np.array([total_sched, total_sets, slowest]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_cover_the_workload(tmp_path):
    import torch.multiprocessing as mp
    from oracle import rta
    from paper_2406_05221_b200 import taskgen
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    per_rank, world = 700, 2
    mp.spawn(_worker, args=(world, port, per_rank, str(tmp_path)), nprocs=world, join=True)
    w = taskgen.WORKLOADS["sweep"]
    whole = w.generate(0, per_rank * world, stream=1)
    wcrt, sched, _ = rta.analyse(whole, rta.POLICY_GCAPS, w.timeslice_us, w.overhead_us)
    parts = np.concatenate([np.load(tmp_path / ("wcrt_%d.npy" % r)) for r in range(world)])
    assert np.array_equal(parts, wcrt)
    totals = np.load(tmp_path / "totals.npy")
    assert totals.tolist() == [float((sched == 1).sum()), float(per_rank * world), float(world)]
