"""The multi-GPU leg of bench.py runs independent replicas (the operator has no exchange step); what the
ranks share is the timing rule: the job is as fast as its slowest rank.  Checked here with two gloo ranks
on the CPU."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, results):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        slowest = bench.max_over_ranks(mine, dist, torch.device("cpu"))
        results[rank] = (slowest, bench.replica_throughput(world, 2.0e12, slowest))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_aggregate_throughput():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        results = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, results), nprocs=world, join=True)
        got = dict(results)
    assert set(got) == {0, 1}
    for rank in range(world):
        slowest, tflops = got[rank]
        assert slowest == pytest.approx(15.0)
        # two replicas of 2 TFLOP each in 15 ms
        assert tflops == pytest.approx(2 * 2.0e12 / 15e-3 / 1e12)


def test_single_process_path_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, torch.device("cpu")) == 3.5
    assert bench.replica_throughput(1, 1.0e12, 1000.0) == pytest.approx(1.0)
