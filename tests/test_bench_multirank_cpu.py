"""The N > 1 path of bench.py is "replicas only": no collective touches the data, the ranks only
agree on the slowest time.  That aggregation is covered here with two gloo ranks on the CPU."""
import os
import sys

import pytest
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
    local_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
    slowest = bench.max_over_ranks(local_ms, world, "cpu")
    out[rank] = (slowest, bench.job_tflops(3.0e12, world, slowest))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation_takes_the_slowest_rank():
    world, port = 2, 29000 + os.getpid() % 1000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1]
        slowest, tflops = out[0]
        assert slowest == 15.0
        assert tflops == pytest.approx(2 * 3.0e12 / 15.0e-3 / 1e12)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, 1, "cpu") == 7.5
    assert bench.method_flops(128, 64, 16, 2) == 6.0 * 128 * 64 * 16 + 3 * 128 * 256 + 6.0 * 112 * 64 * 16 + 3 * 112 * 256
