"""Seeded random plans of every kernel family against the oracle (GPU).

Dimension, radius, shape, boundary, element type, grid extents and step count are drawn at random, the
plan is the default one (the route the library picks by itself), and every output point is compared with
the oracle.  The extents mix ragged sizes with the widths the selection rules switch at."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_21157_b200 import binding as b
from paper_2608_21157_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _draw(rng):
    ndim = int(rng.choice([2, 3]))
    f64 = bool(rng.random() < 0.35)
    box = bool(rng.random() < 0.4)
    if ndim == 3:
        R = int(rng.integers(1, 3 if box else 5))
        nx = int(rng.choice([int(rng.integers(8, 700)), int(rng.choice([128, 256, 384, 512, 640, 132, 260])),
                             4 * int(rng.integers(4, 150))]))
        dims = (int(rng.integers(2 * R + 1, 90)), int(rng.integers(2 * R + 1, 200)), nx)
    else:
        R = int(rng.integers(1, 4 if box else 6))
        nx = int(rng.choice([int(rng.integers(8, 3000)), 4 * int(rng.integers(8, 700)), int(rng.choice([128, 1024, 2048]))]))
        dims = (int(rng.integers(2 * R + 1, 900)), nx)
    steps = int(rng.choice([1, 1, 2, 3, 4, 5, 7, 8]))
    boundary = int(rng.choice([b.ZERO, b.PERIODIC]))
    return ndim, R, box, dims, steps, boundary, (np.float64 if f64 else np.float32)


@pytest.mark.parametrize("seed", [101, 102, 103, 104])
def test_random_default_plans_match_the_oracle(seed):
    rng = np.random.default_rng(seed)
    stream = torch.cuda.current_stream().cuda_stream
    for it in range(40):
        ndim, R, box, dims, steps, boundary, dt = _draw(rng)
        w = (wl.random_box_weights if box else wl.random_star_weights)(ndim, R, 1000 * seed + it, dt)
        a = wl.normal_field(dims, 2000 * seed + it, dt)
        src = torch.from_numpy(a).cuda()
        dst = torch.full_like(src, float("nan"))
        with b.Plan(dims, R, b.BOX if box else b.STAR, w, boundary) as p:
            what = f"dims={dims} R={R} {'box' if box else 'star'} boundary={boundary} {np.dtype(dt).name} " \
                   f"steps={steps} variant={p.variant} fuse={p.get(b.KEY_FUSE_STEPS)}"
            p.apply(src, dst, steps, stream)
            assert p.query_status() == b.OK, what
        got = dst.cpu().numpy()
        assert not np.isnan(got).any(), f"{what}: some output points were never written"
        want = oracle.apply(a, w, boundary, steps)
        tol = wl.tolerance(w, float(np.abs(a).max()), steps)
        err = float(np.max(np.abs(got - want)))
        assert err <= tol, f"{what}: max err {err:.3e} > tol {tol:.3e}"
