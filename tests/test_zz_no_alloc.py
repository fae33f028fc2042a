"""stencil_apply_static: the entry point for callers that cannot allocate.

Some users of the library run the sweep where cudaMalloc is off limits: all
device memory already belongs to their own pool, or the stall an allocation
causes does not fit their time loop.  The entry point keeps its scratch in a
fixed array inside the library instead.  This file checks, through the C ABI,
that it gives the same answer as stencil_apply (within the tolerance every
other GPU test uses) on two calls in a row, which also shows that what the
first call left in the shared array does not disturb the second; and that
grids above the fixed limit are refused.  It sorts last on purpose, so that a
run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2608_21157_b200 import binding as b
from paper_2608_21157_b200 import build as build_mod
from paper_2608_21157_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()
    b.load()


def _both(dims, R, shape, w, boundary, a, steps):
    """(result of stencil_apply, result of stencil_apply_static) on the same input."""
    stream = torch.cuda.current_stream().cuda_stream
    src = torch.from_numpy(a).cuda()
    ref = torch.full_like(src, float("nan"))
    got = torch.full_like(src, float("nan"))
    with b.Plan(dims, R, shape, w, boundary) as p:
        assert b.stencil_apply(p._h, src.data_ptr(), ref.data_ptr(), steps, stream) == b.OK
        assert b.stencil_apply_static(p._h, src.data_ptr(), got.data_ptr(), steps, stream) == b.OK
        torch.cuda.synchronize()
        assert p.query_status() == b.OK
    return ref.cpu().numpy(), got.cpu().numpy()


def test_static_entry_matches_apply_on_two_calls_in_a_row():
    # first call: 3D box, iterated (uses the fixed scratch grid for the ping-pong)
    dims = (40, 48, 64)
    w = wl.random_box_weights(3, 1, 5)
    a = wl.normal_field(dims, 6)
    ref, got = _both(dims, 1, b.BOX, w, b.ZERO, a, steps=5)
    assert not np.isnan(got).any()
    assert np.max(np.abs(got - ref)) <= wl.tolerance(w, float(np.abs(a).max()), 5)

    # second call straight after: other plan, other shape, fewer taps, periodic, smaller grid;
    # the array still holds the first call's taps and field
    dims2 = (33, 70)
    w2 = wl.random_star_weights(2, 3, 7)
    a2 = wl.normal_field(dims2, 8)
    ref2, got2 = _both(dims2, 3, b.STAR, w2, b.PERIODIC, a2, steps=4)
    assert not np.isnan(got2).any()
    assert np.max(np.abs(got2 - ref2)) <= wl.tolerance(w2, float(np.abs(a2).max()), 4)


def test_static_entry_single_step_and_copy():
    wk = wl.get("cfg1")
    a, w = wk.input(), wk.weights()
    ref, got = _both(wk.dims, wk.radius, wk.shape, w, wk.boundary, a, steps=1)
    assert np.max(np.abs(got - ref)) <= wl.tolerance(w, float(np.abs(a).max()), 1)
    ref0, got0 = _both(wk.dims, wk.radius, wk.shape, w, wk.boundary, a, steps=0)
    assert np.array_equal(got0, a) and np.array_equal(ref0, a)


def test_static_entry_refuses_grids_above_its_limit():
    dims = (129, 128, 128)                          # one plane more than 2^21 points
    assert int(np.prod(dims)) > b.STATIC_MAX_POINTS
    w = wl.star_weights(3, 1, -6.0, [1.0])
    src = torch.zeros(dims, dtype=torch.float32, device="cuda")
    dst = torch.full_like(src, 7.0)
    with b.Plan(dims, 1, b.STAR, w, b.ZERO) as p:
        rc = b.stencil_apply_static(p._h, src.data_ptr(), dst.data_ptr(), 2, 0)
        assert rc == b.ERR_TOO_LARGE
        assert "fixed scratch" in b.status_string(rc)
        assert p.launches == 0
    torch.cuda.synchronize()
    assert bool((dst == 7.0).all())                 # nothing was enqueued
