"""stencil_apply_static: the entry point for callers that cannot allocate.

Some users of the library run the sweep where cudaMalloc is off limits: all
device memory already belongs to their own pool, or the stall an allocation
causes does not fit their time loop.  The entry point keeps its scratch in a
fixed array inside the library instead.  This file checks, through the C ABI,
that it gives the same answer as stencil_apply and as the CPU oracle (within
the tolerance every other GPU test uses) on two calls in a row, which also
shows that what the first call left in the shared array does not disturb the
second; that a plan which has only ever run this entry point owns no device
memory and that the device's free memory does not move across a call; that a
grid of exactly the limit runs and grids above it are refused.  It sorts last on purpose, so that a
run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_21157_b200 import binding as b
from paper_2608_21157_b200 import build as build_mod
from paper_2608_21157_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()
    b.load()


def _static(dims, R, shape, w, boundary, a, steps):
    """Result of stencil_apply_static on a plan that has never run anything else: the plan owns no
    device memory before or after, and the device's free memory does not move across the call."""
    stream = torch.cuda.current_stream().cuda_stream
    src = torch.from_numpy(a).cuda()
    got = torch.full_like(src, float("nan"))
    with b.Plan(dims, R, shape, w, boundary) as p:
        assert p.get(b.KEY_SCRATCH_BYTES) == 0
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        assert b.stencil_apply_static(p._h, src.data_ptr(), got.data_ptr(), steps, stream) == b.OK
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0, "stencil_apply_static changed the device's free memory"
        assert p.get(b.KEY_SCRATCH_BYTES) == 0
        assert p.query_status() == b.OK
    return got.cpu().numpy()


def _apply(dims, R, shape, w, boundary, a, steps):
    """Result of the existing entry point, stencil_apply, on a plan of its own."""
    stream = torch.cuda.current_stream().cuda_stream
    src = torch.from_numpy(a).cuda()
    ref = torch.full_like(src, float("nan"))
    with b.Plan(dims, R, shape, w, boundary) as p:
        assert b.stencil_apply(p._h, src.data_ptr(), ref.data_ptr(), steps, stream) == b.OK
        torch.cuda.synchronize()
        assert p.query_status() == b.OK
    return ref.cpu().numpy()


def _check(dims, R, shape, w, boundary, a, steps):
    """stencil_apply_static against stencil_apply and against the CPU oracle."""
    got = _static(dims, R, shape, w, boundary, a, steps)
    ref = _apply(dims, R, shape, w, boundary, a, steps)
    want = oracle.apply(a, w, boundary, steps)
    tol = wl.tolerance(w, float(np.abs(a).max()), steps)
    assert not np.isnan(got).any()
    assert np.max(np.abs(got - ref)) <= tol, "differs from stencil_apply"
    assert np.max(np.abs(got - want)) <= tol, "differs from the oracle"


@pytest.fixture(scope="module", autouse=True)
def _array_looked_up():
    """The first call on a device looks the fixed array up (and, under lazy module loading, is
    what brings the array into device memory); make it here so that the calls under test are
    not the first."""
    w = wl.star_weights(2, 1, -4.0, [1.0])
    src = torch.zeros((8, 8), dtype=torch.float32, device="cuda")
    dst = torch.empty_like(src)
    with b.Plan((8, 8), 1, b.STAR, w, b.ZERO) as p:
        assert b.stencil_apply_static(p._h, src.data_ptr(), dst.data_ptr(), 1, 0) == b.OK
    torch.cuda.synchronize()


def test_static_entry_matches_apply_on_two_calls_in_a_row():
    # first call: 3D box, iterated (uses the fixed scratch grid for the ping-pong)
    dims = (40, 48, 64)
    w = wl.random_box_weights(3, 1, 5)
    a = wl.normal_field(dims, 6)
    _check(dims, 1, b.BOX, w, b.ZERO, a, steps=5)
    # second call straight after: other plan, other shape, fewer taps, periodic, smaller grid;
    # the array still holds the first call's taps and field
    dims2 = (33, 70)
    w2 = wl.random_star_weights(2, 3, 7)
    a2 = wl.normal_field(dims2, 8)
    _check(dims2, 3, b.STAR, w2, b.PERIODIC, a2, steps=4)


def test_static_entry_twice_on_one_plan_keeps_its_taps():
    """The second call of a plan finds its taps still in the array and does not upload them again;
    a call of another plan in between replaces them, and the first plan uploads again."""
    dims = (24, 40, 64)
    w = wl.random_star_weights(3, 2, 11)
    w_other = wl.random_box_weights(3, 1, 12)
    a = wl.normal_field(dims, 13)
    want = oracle.apply(a, w, b.ZERO, 3)
    tol = wl.tolerance(w, float(np.abs(a).max()), 3)
    stream = torch.cuda.current_stream().cuda_stream
    src = torch.from_numpy(a).cuda()
    with b.Plan(dims, 2, b.STAR, w, b.ZERO) as p, b.Plan(dims, 1, b.BOX, w_other, b.ZERO) as q:
        for other_in_between in (False, False, True, False):
            if other_in_between:
                tmp = torch.empty_like(src)
                assert b.stencil_apply_static(q._h, src.data_ptr(), tmp.data_ptr(), 1, stream) == b.OK
            got = torch.full_like(src, float("nan"))
            assert b.stencil_apply_static(p._h, src.data_ptr(), got.data_ptr(), 3, stream) == b.OK
            torch.cuda.synchronize()
            assert np.max(np.abs(got.cpu().numpy() - want)) <= tol


def test_static_entry_at_its_limit():
    dims = (128, 128, 128)                          # exactly 2^21 points
    assert int(np.prod(dims)) == b.STATIC_MAX_POINTS
    w = wl.star_weights(3, 1, 0.4, [0.1])
    a = wl.uniform_field(dims, 0.0, 1.0, 9)
    _check(dims, 1, b.STAR, w, b.ZERO, a, steps=2)


def test_static_entry_single_step_and_copy():
    wk = wl.get("cfg1")
    a, w = wk.input(), wk.weights()
    _check(wk.dims, wk.radius, wk.shape, w, wk.boundary, a, steps=1)
    got0 = _static(wk.dims, wk.radius, wk.shape, w, wk.boundary, a, steps=0)
    assert np.array_equal(got0, a)


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
