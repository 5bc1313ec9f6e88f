"""The multi-rank bookkeeping of bench.py (replicas only, no data-path collective), run as two gloo
ranks on CPU: the timing that is reported is the slowest rank's, and the job-level value counts the
layers of every replica."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = [3.0, 5.5][rank]                                   # each rank timed its own replica
    slowest = bench.max_over_ranks(ms, dist, "cpu")
    dist.barrier()
    out[rank] = slowest
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_rank():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1] == 5.5


def test_whole_job_value_counts_every_replica():
    sys.path.insert(0, ROOT)
    import bench
    one = bench.whole_job_us_per_layer(0.070, 7, 1)        # 70 us per step of 7 layers on one GPU
    two = bench.whole_job_us_per_layer(0.070, 7, 2)        # two replicas, same step time: twice the layers
    assert one == pytest.approx(10.0) and two == pytest.approx(5.0)
    assert bench.max_over_ranks(1.25, None, "cpu") == 1.25
