"""The multi-GPU mode of the benchmark is N independent replicas (the path has no exchange step): the only
cross-rank logic is the max-over-ranks of the timings and the whole-job value.  Checked here with two gloo
ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [100.0 + 10 * rank, 5.0 - rank, 7.0]            # rank 1 is slower on the first, faster on the second
        got = bench.max_over_ranks(mine, dist, "cpu")
        dist.barrier()
        out[rank] = got
    finally:
        dist.destroy_process_group()


def test_max_over_two_gloo_ranks_and_replica_value():
    sys.path.insert(0, ROOT)
    import bench
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29591, out), nprocs=world, join=True)
        assert out[0] == out[1] == [110.0, 5.0, 7.0]
    # two replicas finishing one layer each in 110 us deliver a layer every 55 us
    assert bench.replica_value(110.0, 2) == 55.0
    assert bench.max_over_ranks([1.0, 2.0], None, "cpu") == [1.0, 2.0]
