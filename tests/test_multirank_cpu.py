"""The multi-rank bookkeeping of bench.py (replicas only: a barrier, the max of the ranks' step
times, work summed over ranks) on two gloo ranks on the CPU."""
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
    dist.barrier()
    ms = bench.max_over_ranks(2.0 + rank, dist, torch.device("cpu"))     # ranks took 2 ms and 3 ms
    out[rank] = (ms, bench.aggregate_value(6e9, ms, world))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_work():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert out[0][0] == out[1][0] == 3.0
        assert abs(out[0][1] - 2 * 6e9 / 3e-3 / 1e12) < 1e-9


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.5, None, None) == 1.5
    assert bench.aggregate_value(1e12, 1000.0, 1) == 1.0
