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


# ---------------------------------------------------------------- slab decomposition --
def test_slab_ranges_cover_the_axis_once():
    from paper_2608_21157_b200.sharded import slab_range
    for n, world in [(512, 8), (10, 3), (7, 7), (100, 6)]:
        edges = [slab_range(n, world, r) for r in range(world)]
        assert edges[0][0] == 0 and edges[-1][1] == n
        assert all(edges[r][1] == edges[r + 1][0] for r in range(world - 1))
        sizes = [b - a for a, b in edges]
        assert max(sizes) - min(sizes) <= 1


def _sharded_worker(rank, world, port, dims, R, steps, halo_steps, overlap, periodic, out):
    import numpy as np
    import oracle
    from paper_2608_21157_b200 import workloads as wl
    from paper_2608_21157_b200.sharded import ShardedSweep
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ndim = len(dims)
        w = wl.random_box_weights(ndim, R, 5)
        a = wl.normal_field(dims, 6)                    # every rank builds the same global field

        calls = []
        boundary = oracle.PERIODIC if periodic else oracle.ZERO

        def local_apply(src, dst, nsteps):              # sweeps of the local slab, on the CPU
            calls.append(nsteps)
            dst.copy_(torch.from_numpy(oracle.apply(src.numpy(), w, boundary, nsteps)))

        ranges = []

        def local_apply_planes(src, dst, z_begin, z_end):   # one sweep, output planes [z_begin, z_end) only
            ranges.append((z_begin, z_end))
            full = torch.from_numpy(oracle.apply(src.numpy(), w, boundary, 1))
            dst[z_begin:z_end].copy_(full[z_begin:z_end])

        sw = ShardedSweep(dims, R, 1, w, 1 if periodic else 0, rank=rank, world=world, dist=dist,
                          halo_steps=halo_steps, local_apply=local_apply,
                          local_apply_planes=local_apply_planes if overlap else None)
        assert sw.overlap == (overlap and halo_steps == 1)
        expected_ghosts = halo_steps * R * (2 if periodic else (rank > 0) + (rank < world - 1))
        assert sw.local_dims[0] == (sw.z1 - sw.z0) + expected_ghosts
        ext = sw.scatter(torch.from_numpy(a))
        res = sw.apply(ext, steps)
        if sw.overlap:
            # per step: the planes that read no ghost plane first, then R planes per neighbour; together
            # they cover the own planes exactly once
            per_step = 3 if periodic else 1 + (rank > 0) + (rank < world - 1)
            assert len(ranges) == steps * per_step and not calls
            covered = sorted(ranges[:per_step])
            assert covered[0][0] == sw.lo and covered[-1][1] == sw.lo + sw.nlocal
            assert all(covered[i][1] == covered[i + 1][0] for i in range(per_step - 1))
            calls = [1] * steps
        out[rank] = (sw.z0, sw.z1, sw.interior(res).numpy().copy(), list(calls))
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(180)
@pytest.mark.parametrize("world,dims,R,steps,halo_steps,overlap,periodic", [
    (2, (11, 9, 12), 1, 3, 1, False, False), (3, (13, 10), 2, 4, 1, False, False), (2, (4, 6, 8), 2, 2, 1, False, False),
    (2, (11, 9, 12), 1, 5, 2, False, False),      # two steps per exchange, the last round one step
    (3, (19, 10), 2, 6, 3, False, False),         # three ranks, ghost zones of 6 rows, two rounds
    (2, (12, 6, 8), 1, 4, 4, False, False),       # one exchange for the whole run
    (3, (17, 9, 12), 1, 3, 1, True, False),       # exchange overlapped with the sweep of the inner planes
    (2, (14, 6, 8), 2, 2, 1, True, False),
    (2, (11, 9, 12), 1, 4, 2, True, False),       # overlap asked for, but two steps per exchange: not used
    (3, (13, 9, 12), 1, 3, 1, False, True),       # periodic: the ranks form a ring, ghosts on both sides of every rank
    (2, (11, 10), 2, 5, 2, False, True),          # a ring of two: both neighbours are the same peer
    (2, (12, 6, 8), 1, 4, 4, False, True),
    (3, (17, 9, 12), 1, 3, 1, True, True),        # ... with the exchange overlapped
])
def test_sharded_sweep_equals_the_single_grid_sweep(world, dims, R, steps, halo_steps, overlap, periodic):
    """Halo exchange + local sweeps on 2-3 gloo ranks reproduce the sweep of the whole grid
    bit for bit (every point sees the same neighbours in the same order), also when the
    ghost zones are deep enough for several steps between two exchanges."""
    import numpy as np
    import oracle
    from paper_2608_21157_b200 import workloads as wl
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_sharded_worker, args=(world, port, dims, R, steps, halo_steps, overlap, periodic, out),
                 nprocs=world, join=True)
        parts = dict(out)
    w = wl.random_box_weights(len(dims), R, 5)
    a = wl.normal_field(dims, 6)
    want = oracle.apply(a, w, oracle.PERIODIC if periodic else oracle.ZERO, steps)
    got = np.empty_like(want)
    for r in range(world):
        z0, z1, block, calls = parts[r]
        got[z0:z1] = block
        assert sum(calls) == steps and len(calls) == -(-steps // halo_steps) and max(calls) <= halo_steps
    assert np.array_equal(got, want)


# ------------------------------------------------------ the benchmark's sharded arm --
def _sharded_bench_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        total = 0.0
        for my_ms in ([4.0, 6.0] if rank == 0 else [5.0, 5.5]):     # two timed applies: the slower rank differs
            dist.barrier()
            total += bench.max_over_ranks(my_ms, dist, torch.device("cpu"))
        out[rank] = (total, bench.sharded_job_summary((512, 512, 512), 1, 16, 2, 2, total, world, 4))
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_sharded_arm_counts_the_grid_once_over_the_slowest_rank():
    """`bench.py --sharded`: all ranks share ONE grid, so the job's value is the grid's
    point-updates over the sum of the slowest rank's times, not world x that (the replicas rule)."""
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_sharded_bench_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    total, s = res[0]
    assert total == 5.0 + 6.0
    assert s["value"] == pytest.approx(512 ** 3 * 16 * 2 / 11e-3 / 1e9)
    # two steps between exchanges: 8 rounds, each 2 planes of 512 x 512 floats to either neighbour
    assert s["messages_per_rank_per_apply"] == 2 * 8
    assert s["exchange_bytes_per_rank_per_apply"] == 2 * 8 * 2 * 512 * 512 * 4
    assert s["exchange_bytes_per_rank_per_time_step"] == pytest.approx(2 * 512 * 512 * 4)


def test_sharded_arm_on_one_rank_sends_nothing():
    s = bench.sharded_job_summary((64, 32, 128), 2, 5, 2, 3, 10.0, 1, 4)
    assert s["exchange_bytes_per_rank_per_apply"] == 0 and s["messages_per_rank_per_apply"] == 0
    assert s["value"] == pytest.approx(64 * 32 * 128 * 5 * 3 / 10e-3 / 1e9)
