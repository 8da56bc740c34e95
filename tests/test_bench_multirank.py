"""The N > 1 path of bench.py shards nothing but the batch: every rank transforms its own 60 examples and
the only exchange is the max-over-ranks of the timings.  This runs that host logic on two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, results):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seconds = 0.5 + 0.25 * rank                      # rank 1 is the slow one
    slowest = bench.max_over_ranks(seconds, world, device="cpu")
    dist.barrier()
    results[rank] = (slowest, bench.whole_job_value(60, 5, slowest, world))
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_whole_job_value():
    world, port = 2, 29512 + os.getpid() % 400
    with mp.Manager() as mgr:
        results = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, results), nprocs=world, join=True)
        assert len(results) == 2
        for rank in range(world):
            slowest, value = results[rank]
            assert slowest == 0.75
            assert value == 2 * 60 * 5 / 0.75


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.25, 1) == 1.25
    assert bench.whole_job_value(60, 5, 0.4, 1) == 60 * 5 / 0.4
