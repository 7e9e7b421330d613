"""The N > 1 path of bench.py on CPU: two gloo ranks, each with its own shard's time; the
job-level number is the whole-job work over the slowest rank's time."""
import os
import sys

import pytest
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
        mine = 10.0 + 5.0 * rank                      # rank 1 is the slower replica
        slowest = bench.max_over_ranks(mine, world)
        dist.barrier()
        out[rank] = (slowest, bench.whole_job_tops(slowest, world))
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_replica_and_the_whole_job():
    sys.path.insert(0, ROOT)
    import bench
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        slowest, tops = res[rank]
        assert slowest == pytest.approx(15.0)
        assert tops == pytest.approx(2 * bench.OPS_PER_STEP / 15e-3 / 1e12)
    # one rank: nothing to reduce, no process group needed
    assert bench.max_over_ranks(7.0, 1) == 7.0
    assert bench.whole_job_tops(7.0, 1) == pytest.approx(bench.OPS_PER_STEP / 7e-3 / 1e12)
