"""The N > 1 path of bench.py: replicas only, no data-path collective.  What ranks share is the
timing rule -- the job's time is the slowest rank's -- and the whole-job aggregate.  Checked here
with two `gloo` ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        worst = bench.max_over_ranks(mine, world, "cpu")
        out[rank] = (worst, bench.aggregate_tokens_per_s(32, 100, world, worst * 1e-3))
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_aggregate():
    world = 2
    port = 29500 + os.getpid() % 1000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1]
        worst, value = out[0]
        assert worst == 15.0
        assert abs(value - 2 * 32 * 100 / 15e-3) < 1e-6


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
