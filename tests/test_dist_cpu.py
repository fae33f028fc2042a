"""The multi-rank path of the benchmark on CPU (gloo, world_size 2): every rank
runs its own replica, the reported time is the slowest rank's, the value is
the sum of all ranks' points over that time.  No GPU, no data-path collective."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        dist.barrier()
        slowest = bench.max_over_ranks(my_ms, dist, torch.device("cpu"))
        value = bench.whole_job_gpoints(world, 1000, 4, slowest)
        out[rank] = (slowest, value)
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_ranks_report_the_slowest_time_and_the_summed_points():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    slowest, value = res[0]
    assert slowest == 15.0
    assert value == pytest.approx(2 * 1000 * 4 / 15e-3 / 1e9)


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.whole_job_gpoints(1, 2_000_000_000, 1, 1000.0) == pytest.approx(2.0)
