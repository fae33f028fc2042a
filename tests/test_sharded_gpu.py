"""The slab decomposition on real GPUs: two ranks, one GPU each, halo exchange over NCCL, the real
kernels as the local sweep; the gathered result against the CPU oracle's sweep of the whole grid.
Needs two visible GPUs (skipped otherwise); the exchange logic itself is covered on CPU with gloo
ranks in test_dist_cpu.py.  Also the benchmark's sharded arm on one rank."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from paper_2608_21157_b200 import binding as b
from paper_2608_21157_b200 import build as build_mod
from paper_2608_21157_b200 import workloads as wl

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()
    b.load()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _nccl_worker(rank, world, port, dims, R, box, steps, halo_steps, overlap, periodic, out):
    import torch.distributed as dist
    from paper_2608_21157_b200.sharded import ShardedSweep
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(rank)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", rank))
    try:
        w = wl.star_weights(len(dims), 1, 1.0 - 0.2 * len(dims), [0.1]) if not box else wl.random_box_weights(len(dims), R, 5)
        a = wl.uniform_field(dims, 0.0, 1.0, 6)          # every rank builds the same global field
        sw = ShardedSweep(dims, R, b.BOX if box else b.STAR, w, b.PERIODIC if periodic else b.ZERO, rank=rank,
                          world=world, dist=dist, halo_steps=halo_steps, overlap=overlap)
        assert sw.overlap == (overlap and halo_steps == 1 and not periodic)
        ext = sw.scatter(torch.from_numpy(a).cuda())
        res = sw.apply(ext, steps)
        torch.cuda.synchronize()
        assert sw._plan.query_status() == b.OK
        out[rank] = (sw.z0, sw.z1, sw.interior(res).cpu().numpy().copy())
        sw.close()
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
@pytest.mark.parametrize("dims,R,box,steps,halo_steps,overlap,periodic", [
    ((48, 40, 128), 1, False, 5, 1, True, False),      # one step per exchange, overlapped with the inner planes
    ((48, 40, 128), 1, False, 6, 2, False, False),     # two steps per exchange: fused passes on the slabs
    ((40, 36, 128), 1, True, 3, 1, True, False),       # the 27-point box
    ((48, 40, 128), 1, False, 4, 2, False, True),      # periodic: a ring of two
    ((96, 256), 1, False, 8, 4, False, False),         # 2D: rows are the split axis, four fused steps per exchange
], ids=["overlap", "two_steps_per_exchange", "box", "periodic_ring", "2d_fused"])
def test_two_nccl_ranks_reproduce_the_single_grid_sweep(dims, R, box, steps, halo_steps, overlap, periodic):
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two visible GPUs")
    import torch.multiprocessing as mp
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_nccl_worker, args=(world, port, dims, R, box, steps, halo_steps, overlap, periodic, out),
                 nprocs=world, join=True)
        parts = dict(out)
    w = wl.star_weights(len(dims), 1, 1.0 - 0.2 * len(dims), [0.1]) if not box else wl.random_box_weights(len(dims), R, 5)
    a = wl.uniform_field(dims, 0.0, 1.0, 6)
    want = oracle.apply(a, w, b.PERIODIC if periodic else b.ZERO, steps)
    got = np.empty_like(want)
    for r in range(world):
        z0, z1, block = parts[r]
        got[z0:z1] = block
    assert np.max(np.abs(got - want)) <= wl.tolerance(w, 1.0, steps)


@pytest.mark.timeout(300)
def test_sharded_bench_arm_runs_on_one_rank():
    """`bench.py --sharded` with one rank is the plain iterated apply through the sharding layer: the
    line names the strong-scaling arm and counts the grid once."""
    env = dict(os.environ, NCCL_DEBUG="WARN")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--sharded", "--workload", "cfg5",
                        "--dims", "64,64,128", "--steps", "3", "--warmup", "3"], capture_output=True, text=True,
                       env=env, timeout=240)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["scaling"] == "strong" and line["n_gpus"] == 1 and line["gpu_launches"] > 0
    assert line["config"]["halo_steps"] == 2 and line["config"]["exchange_bytes_per_rank_per_time_step"] == 0
    assert line["value"] == pytest.approx(64 * 64 * 128 * 64 / (line["ms_per_step"] / 1e3) / 1e9, rel=1e-3)
