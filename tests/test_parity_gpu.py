"""CUDA path vs CPU oracle, element by element, through the C ABI.

Acceptance: max|gpu - oracle| <= 1e-5 * sum|w| * max|in| * steps + 1e-6.
Every output buffer is poisoned with NaN and fenced by guard bands first, so a
point that was never written or a store outside the grid fails the test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_21157_b200 import binding as b
from paper_2608_21157_b200 import build as build_mod
from paper_2608_21157_b200 import workloads as wl

pytestmark = pytest.mark.gpu

GUARD = 4096          # floats of guard band on each side of the output


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()
    b.load()


def gpu_sweep(dims, R, shape, weights, boundary, a, steps=1, variant=None, repeat=1, **knobs):
    """Runs the library on `a`; returns the result as numpy after checking guards."""
    dev = torch.device("cuda:0")
    n = int(np.prod(dims))
    src = torch.from_numpy(a).to(dev)
    src_copy = src.clone()
    buf = torch.full((n + 2 * GUARD,), float("nan"), dtype=src.dtype, device=dev)
    buf[:GUARD] = 12345.0
    buf[GUARD + n:] = 12345.0
    dst = buf[GUARD:GUARD + n]
    stream = torch.cuda.current_stream().cuda_stream
    with b.Plan(dims, R, shape, weights, boundary, variant=variant, **knobs) as p:
        for _ in range(repeat):
            p.apply(src, dst, steps, stream)
        assert p.query_status() == b.OK
        used = p.variant
    torch.cuda.synchronize()
    assert torch.equal(src, src_copy), "input was modified"
    assert bool((buf[:GUARD] == 12345.0).all()) and bool((buf[GUARD + n:] == 12345.0).all()), \
        "store outside the output grid"
    out = dst.cpu().numpy().reshape(dims)
    assert not np.isnan(out).any(), "some output points were never written"
    return out, used


def check(dims, R, shape, weights, boundary, a, steps=1, **kw):
    got, used = gpu_sweep(dims, R, shape, weights, boundary, a, steps, **kw)
    want = oracle.apply(a, weights, boundary, steps)
    tol = wl.tolerance(weights, float(np.abs(a).max()), steps)
    err = float(np.max(np.abs(got.astype(np.float64) - want.astype(np.float64)))) if got.size else 0.0
    assert err <= tol, f"{used}: max err {err:.3e} > tol {tol:.3e} for dims={dims} R={R} steps={steps} {kw}"
    return used


# ------------------------------------------------------- randomized requests --
def _random_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < n:
        ndim = int(rng.integers(2, 4))
        R = int(rng.choice([1, 1, 1, 2, 2, 3, 4, 5, 6, 8]))
        box = bool(rng.integers(0, 2))
        if box and ndim == 3 and R > 2:
            R = int(rng.integers(1, 3))                 # keep the oracle's tap count small
        if box and R > 4:
            R = 4
        f64 = bool(rng.integers(0, 3) == 0)
        periodic = bool(rng.integers(0, 2))
        steps = int(rng.choice([1, 1, 2, 3, 5, 8]))
        # the fastest axis: mostly 16-byte rows of the widths the tiled and fused kernels distinguish, some odd ones
        nx = int(rng.choice([8, 64, 128, 132, 200, 256, 260, 384, 388, 512, 520, 1000, 61, 130, 255]))
        if ndim == 2:
            ny = int(rng.integers(1, 300))
            dims = (ny, nx)
        else:
            budget = 400_000 // nx
            ny = int(rng.integers(1, max(2, min(60, budget))))
            nz = int(rng.integers(1, max(2, min(60, budget // ny + 1))))
            dims = (nz, ny, nx)
        taps = (2 * R + 1) ** ndim if box else 2 * ndim * R + 1
        if int(np.prod(dims)) * taps * steps > 60_000_000:
            continue
        cases.append((dims, R, box, periodic, steps, f64))
    return cases


@pytest.mark.parametrize("dims,R,box,periodic,steps,f64", _random_cases(90, 20261125))
def test_randomized_requests_match_oracle(dims, R, box, periodic, steps, f64):
    """Seeded random requests through the default route of the library (whatever kernel, fusion
    depth and periodic route it picks for them), every point against the oracle."""
    dt = np.float64 if f64 else np.float32
    nd = len(dims)
    w = (wl.random_box_weights if box else wl.random_star_weights)(nd, R, 7 + R, dt)
    a = wl.normal_field(dims, 11 + steps, dt)
    boundary = b.PERIODIC if periodic else b.ZERO
    got, used = gpu_sweep(dims, R, b.BOX if box else b.STAR, w, boundary, a, steps)
    want = oracle.apply(a, w, boundary, steps)
    tol = wl.tolerance(w, float(np.abs(a).max()), steps)
    err = float(np.max(np.abs(got.astype(np.float64) - want.astype(np.float64))))
    assert err <= tol, f"{used}: {err:.3e} > {tol:.3e} dims={dims} R={R} box={box} periodic={periodic} steps={steps} f64={f64}"


# ------------------------------------------------------------------ generic --
GENERIC_CASES = [
    # dims, R, star?, boundary
    ((256, 256), 1, True, b.ZERO),
    ((5, 7), 1, False, b.ZERO), ((5, 7), 2, False, b.PERIODIC), ((33, 47), 3, False, b.ZERO),
    ((2, 3), 3, False, b.ZERO), ((2, 3), 3, False, b.PERIODIC), ((1, 9), 1, True, b.ZERO),
    ((1, 1), 2, False, b.PERIODIC), ((61, 130), 4, True, b.PERIODIC), ((40, 64), 8, False, b.ZERO),
    ((5, 7, 11), 1, False, b.ZERO), ((5, 7, 11), 2, False, b.PERIODIC), ((3, 2, 4), 4, True, b.ZERO),
    ((19, 23, 30), 1, True, b.PERIODIC), ((17, 33, 66), 2, True, b.ZERO), ((9, 12, 20), 3, False, b.ZERO),
    ((1, 1, 5), 1, False, b.ZERO), ((12, 10, 36), 4, False, b.ZERO),
]


@pytest.mark.parametrize("dims,R,star,boundary", GENERIC_CASES)
def test_generic_kernel_small_and_odd_shapes(dims, R, star, boundary):
    ndim = len(dims)
    w = wl.random_star_weights(ndim, R, 7) if star else wl.random_box_weights(ndim, R, 7)
    a = wl.normal_field(dims, 8)
    used = check(dims, R, b.STAR if star else b.BOX, w, boundary, a, variant=b.VARIANT_GENERIC)
    assert used == "generic"


@pytest.mark.parametrize("steps", [0, 1, 2, 3, 6])
@pytest.mark.parametrize("boundary", [b.ZERO, b.PERIODIC])
def test_generic_iteration_and_ping_pong(steps, boundary):
    dims = (9, 14, 22)
    w = wl.random_box_weights(3, 1, 11)              # sum|w| = 1: iterates stay bounded
    a = wl.normal_field(dims, 12)
    check(dims, 1, b.BOX, w, boundary, a, steps=steps, variant=b.VARIANT_GENERIC)


# ------------------------------------------------------------------- stream --
def _stream_knob_sets(R, box):
    """Every compiled tile shape of the operator (tile_y = rows per thread x consumer warps)."""
    if box and R == 2:
        return [dict(), dict(tile_y=16), dict(tile_y=14), dict(tile_y=8),
                dict(tile_y=16, rows_per_thread=2)]
    if box or R == 1:
        return [dict(), dict(tile_y=16), dict(tile_y=14), dict(tile_y=32), dict(tile_y=28), dict(tile_y=8)]
    if R == 4:
        return [dict(), dict(tile_y=16), dict(tile_y=14), dict(tile_y=32, rows_per_thread=4),
                dict(tile_y=32, rows_per_thread=2)]
    if R == 3:
        return [dict(), dict(tile_y=16), dict(tile_y=14), dict(tile_y=32)]
    return [dict(), dict(tile_y=16), dict(tile_y=14), dict(tile_y=32)]


STREAM_OPS = [(1, False), (2, False), (3, False), (4, False), (1, True), (2, True)]


@pytest.mark.parametrize("R,box", STREAM_OPS)
@pytest.mark.parametrize("dims,chunk_z,stages", [
    ((37, 45, 132), 10, 3),      # ragged in x, y and z; several chunks; 2 x-tiles
    ((8, 16, 128), 0, 0),        # exactly one tile, default knobs
    ((3, 5, 4), 0, 2),           # smaller than one tile and than the stencil reach
    ((70, 33, 260), 32, 0),      # three x-tiles, last one 4 points wide
])
def test_stream_kernel_matches_oracle(R, box, dims, chunk_z, stages):
    w = wl.random_box_weights(3, R, 21) if box else wl.random_star_weights(3, R, 21)
    a = wl.normal_field(dims, 22)
    for knobs in _stream_knob_sets(R, box):
        used = check(dims, R, b.BOX if box else b.STAR, w, b.ZERO, a, variant=b.VARIANT_STREAM,
                     chunk_z=chunk_z or None, stages=stages or None, **knobs)
        assert used == "stream"


@pytest.mark.parametrize("R,box", STREAM_OPS)
@pytest.mark.parametrize("steps", [2, 5])
def test_stream_iteration(R, box, steps):
    dims = (21, 40, 136)
    w = wl.random_box_weights(3, R, 31) if box else wl.random_star_weights(3, R, 31)
    a = wl.normal_field(dims, 32)
    check(dims, R, b.BOX if box else b.STAR, w, b.ZERO, a, steps=steps, variant=b.VARIANT_STREAM)


def test_stream_streaming_store_and_determinism():
    dims = (40, 50, 256)
    w = wl.fd8_laplacian_weights(3)
    a = wl.smooth_sine_field(dims, 4)
    one, _ = gpu_sweep(dims, 4, b.STAR, w, b.ZERO, a, variant=b.VARIANT_STREAM, streaming_store=1)
    two, _ = gpu_sweep(dims, 4, b.STAR, w, b.ZERO, a, variant=b.VARIANT_STREAM, repeat=3)
    assert np.array_equal(one, two)                 # same summation order, bitwise repeatable
    want = oracle.apply(a, w, b.ZERO, 1)
    assert np.max(np.abs(one - want)) <= wl.tolerance(w, float(np.abs(a).max()), 1)


def test_time_composition_on_gpu():
    dims = (24, 32, 64)
    w = wl.star_weights(3, 1, 0.4, [0.1])
    a = wl.uniform_field(dims, 0.0, 1.0, 41)
    full, _ = gpu_sweep(dims, 1, b.STAR, w, b.ZERO, a, steps=7)
    half, _ = gpu_sweep(dims, 1, b.STAR, w, b.ZERO, a, steps=3)
    rest, _ = gpu_sweep(dims, 1, b.STAR, w, b.ZERO, half, steps=4)
    assert np.max(np.abs(full - rest)) <= wl.tolerance(w, 1.0, 7)


def test_apply_host_round_trip():
    wk = wl.get("cfg2").scaled((40, 48, 128))       # too few planes for slabs: one upload, one sweep
    a = wk.input()
    w = wk.weights()
    src = torch.from_numpy(a).pin_memory()
    dst = torch.empty_like(src).pin_memory()
    with b.Plan.for_workload(wk) as p:
        p.apply_host(src, dst, 1, torch.cuda.current_stream().cuda_stream)
        assert p.launches == 1
        assert p.get(b.KEY_SCRATCH_BYTES) == 2 * a.nbytes
    want = oracle.apply(a, w, b.ZERO, 1)
    assert np.max(np.abs(dst.numpy() - want)) <= wl.tolerance(w, float(np.abs(a).max()), 1)


@pytest.mark.parametrize("name,dims", [("cfg2", (100, 48, 128)), ("cfg4", (75, 40, 132)), ("cfg3", (64, 33, 128))])
@pytest.mark.parametrize("pinned,in_place", [(True, False), (False, False), (True, True)])
def test_apply_host_pipelined_slabs(name, dims, pinned, in_place):
    """Enough planes for the slab pipeline (upload / sweep / download overlapped): slab seams
    need the halo planes of the next slab, and an in-place host buffer must survive."""
    wk = wl.get(name).scaled(dims)
    a, w = wk.input(), wk.weights()
    want = oracle.apply(a, w, b.ZERO, 1)
    src = torch.from_numpy(a.copy())
    if pinned:
        src = src.pin_memory()
    dst = src if in_place else torch.full_like(src, float("nan"))
    if pinned and not in_place:
        dst = dst.pin_memory()
    with b.Plan.for_workload(wk) as p:
        for _ in range(2):                           # second call reuses streams, events, grids
            if in_place:
                src.copy_(torch.from_numpy(a))
            p.apply_host(src, dst, 1, torch.cuda.current_stream().cuda_stream)
        assert p.launches == 16                      # 8 slabs per call
        assert p.query_status() == b.OK
    assert np.max(np.abs(dst.numpy() - want)) <= wl.tolerance(w, float(np.abs(a).max()), 1)


def test_non_default_stream():
    dims = (16, 32, 128)
    w = wl.random_box_weights(3, 1, 51)
    a = wl.normal_field(dims, 52)
    s = torch.cuda.Stream()
    src = torch.from_numpy(a).cuda()
    dst = torch.empty_like(src)
    torch.cuda.synchronize()
    with b.Plan(dims, 1, b.BOX, w, b.ZERO) as p:
        with torch.cuda.stream(s):
            p.apply(src, dst, 3, s.cuda_stream)
        s.synchronize()
        assert p.launches == 3
    want = oracle.apply(a, w, b.ZERO, 3)
    assert np.max(np.abs(dst.cpu().numpy() - want)) <= wl.tolerance(w, float(np.abs(a).max()), 3)


@pytest.mark.parametrize("R", [5, 6, 7, 8])
@pytest.mark.parametrize("dims,chunk_z,stages", [
    ((37, 45, 132), 10, 3),      # ragged in x, y and z; several chunks; 2 x-tiles
    ((8, 16, 128), 0, 0),        # exactly one tile
    ((3, 5, 4), 0, 2),           # much smaller than the stencil reach
    ((40, 33, 260), 0, 0),       # three x-tiles, the last 4 points wide
])
def test_wide_star_stream_kernel_matches_oracle(R, dims, chunk_z, stages):
    """Stars of radius 5..8 on the tiled 3D kernel (8-column halos, one row per thread)."""
    w = wl.random_star_weights(3, R, 23)
    a = wl.normal_field(dims, 24)
    for knobs in (dict(), dict(tile_y=8)):
        used = check(dims, R, b.STAR, w, b.ZERO, a, variant=b.VARIANT_STREAM, chunk_z=chunk_z or None,
                     stages=stages or None, **knobs)
        assert used == "stream"
    used = check(dims, R, b.STAR, w, b.ZERO, a, steps=3)
    assert used == "stream"
    if min(dims) >= 2 * R:
        used = check(dims, R, b.STAR, w, b.PERIODIC, a, steps=2)         # wrap correction is the only route here
        assert used == "stream"


@pytest.mark.parametrize("R", [5, 6, 7, 8])
@pytest.mark.parametrize("dims,chunk,stages", [((67, 132), 0, 0), ((200, 260), 37, 2), ((3, 8), 0, 0), ((129, 512), 16, 4)])
def test_wide_star_rows2d_kernel_matches_oracle(R, dims, chunk, stages):
    """Stars of radius 5..8 on the 2D row-streaming kernel (8-column halos)."""
    w = wl.random_star_weights(2, R, 25)
    a = wl.normal_field(dims, 26)
    used = check(dims, R, b.STAR, w, b.ZERO, a, chunk_z=chunk or None, stages=stages or None)
    assert used == "stream"
    used = check(dims, R, b.STAR, w, b.ZERO, a, steps=3)
    assert used == "stream"
    if min(dims) >= 2 * R:
        used = check(dims, R, b.STAR, w, b.PERIODIC, a, steps=2)
        assert used == "stream"


@pytest.mark.parametrize("R", [5, 6, 7, 8])
@pytest.mark.parametrize("dims,chunk,stages", [((67, 66), 0, 0), ((200, 258), 37, 2), ((3, 8), 0, 0), ((40, 33, 130), 0, 0),
                                               ((37, 29, 64), 9, 3), ((3, 5, 4), 0, 2)])
def test_wide_star_fp64_kernels_match_oracle(R, dims, chunk, stages):
    """FP64 stars of radius 5..8 on the tiled kernels (8 halo doubles per side)."""
    nd = len(dims)
    w = wl.random_star_weights(nd, R, 27, np.float64)
    a = wl.normal_field(dims, 28, np.float64)
    for steps in (1, 3):
        got, used = gpu_sweep(dims, R, b.STAR, w, b.ZERO, a, steps, chunk_z=chunk or None, stages=stages or None)
        assert used == "stream" and got.dtype == np.float64
        want = oracle.apply(a, w, b.ZERO, steps)
        assert float(np.max(np.abs(got - want))) <= wl.tolerance(w, float(np.abs(a).max()), steps)
    if min(dims) >= 2 * R:
        got, used = gpu_sweep(dims, R, b.STAR, w, b.PERIODIC, a, 2)
        assert used == "stream"
        want = oracle.apply(a, w, b.PERIODIC, 2)
        assert float(np.max(np.abs(got - want))) <= wl.tolerance(w, float(np.abs(a).max()), 2)


@pytest.mark.parametrize("dims,R,box,steps", [
    ((32, 40, 128), 1, False, 1), ((32, 40, 128), 1, False, 4), ((20, 30, 256), 3, False, 2),
    ((33, 50, 128), 1, True, 2), ((40, 260), 2, False, 3), ((64, 256), 1, True, 5),
])
def test_apply_host_on_periodic_plans(dims, R, box, steps):
    """The host-buffer entry point takes the same periodic routes as the device one."""
    nd = len(dims)
    w = (wl.random_box_weights if box else wl.random_star_weights)(nd, R, 5)
    a = wl.normal_field(dims, 6)
    src = torch.from_numpy(a).pin_memory()
    dst = torch.empty_like(src).pin_memory()
    with b.Plan(dims, R, b.BOX if box else b.STAR, w, b.PERIODIC) as p:
        p.apply_host(src, dst, steps, torch.cuda.current_stream().cuda_stream)
        assert p.query_status() == b.OK
    want = oracle.apply(a, w, b.PERIODIC, steps)
    assert float(np.max(np.abs(dst.numpy() - want))) <= wl.tolerance(w, float(np.abs(a).max()), steps)


# ------------------------------------- periodic boundary wrapped inside the sweep --
@pytest.mark.parametrize("R", [1, 2, 3, 4])
@pytest.mark.parametrize("dims,chunk_z,knobs", [
    ((19, 37, 128), 0, {}),                       # one tile per row: it touches both x faces
    ((12, 50, 384), 5, {}),                       # three tiles per row, several z chunks, ragged last tile in y
    ((9, 16, 256), 0, {}),                        # one tile in y at the default tile height: both y faces
    ((8, 8, 128), 3, {}),                         # every extent exactly 2R for radius 4
    ((21, 33, 256), 4, dict(tile_y=14)),          # the 7-warp tiles
    ((10, 70, 128), 0, dict(rows_per_thread=4)),  # 32-row tiles
    ((11, 21, 64), 4, {}),                        # FP64: one 64-column tile per row
    ((7, 40, 192), 0, {}),                        # FP64: three tiles per row (fp32 takes another route here)
])
@pytest.mark.parametrize("f64", [False, True])
def test_periodic_3d_star_wrapped_inside_the_sweep(R, dims, chunk_z, knobs, f64):
    """Periodic 3D stars on rows of whole tiles: the sweep wraps x, y and z itself (one launch per step,
    no correction kernel, no padded copy); fused passes are switched off to reach it for radius 1."""
    if min(dims) < 2 * R:
        pytest.skip("needs every extent >= 2R")
    if f64 and knobs:
        pytest.skip("the tile-shape knobs belong to the fp32 kernel")
    dt = np.float64 if f64 else np.float32
    w = wl.random_star_weights(3, R, 81, dt)
    a = wl.normal_field(dims, 82, dt)
    for steps in (1, 3):
        dev = torch.device("cuda:0")
        src = torch.from_numpy(a).to(dev)
        dst = torch.full_like(src, float("nan"))
        try:
            plan = b.Plan(dims, R, b.STAR, w, b.PERIODIC, fuse_steps=1, chunk_z=chunk_z or None, **knobs)
        except b.StencilError as e:                    # a tile shape this radius does not have
            assert e.status == b.ERR_UNSUPPORTED and knobs
            return
        with plan as p:
            p.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)
            assert p.query_status() == b.OK
            if dims[-1] % (64 if f64 else 128) == 0:
                assert p.launches == steps and p.get(b.KEY_SCRATCH_BYTES) == (a.nbytes if steps > 1 else 0)
        got = dst.cpu().numpy()
        want = oracle.apply(a, w, b.PERIODIC, steps)
        tol = wl.tolerance(w, float(np.abs(a).max()), steps)
        err = float(np.max(np.abs(got - want)))
        assert err <= tol, f"R={R} dims={dims} steps={steps} f64={f64}: {err:.3e} > {tol:.3e}"


@pytest.mark.parametrize("R", [1, 2])
@pytest.mark.parametrize("dims,chunk_z,knobs", [
    ((11, 23, 128), 0, {}),                       # one tile per row: all four corners in one tile
    ((9, 40, 384), 4, {}),                        # three tiles per row, ragged last tile in y
    ((6, 16, 256), 0, {}),                        # one tile in y
    ((7, 30, 256), 3, dict(tile_y=14)),
    ((5, 37, 128), 0, dict(rows_per_thread=1)),
    ((9, 19, 64), 2, {}),                         # FP64: one 64-column tile per row
])
@pytest.mark.parametrize("f64", [False, True])
def test_periodic_3d_box_wrapped_inside_the_sweep(R, dims, chunk_z, knobs, f64):
    """Periodic 3D boxes on rows of whole tiles: the sweep wraps x, y and z itself, corners of the halo included."""
    if f64 and knobs:
        pytest.skip("the tile-shape knobs belong to the fp32 kernel")
    dt = np.float64 if f64 else np.float32
    w = wl.random_box_weights(3, R, 83, dt)
    a = wl.normal_field(dims, 84, dt)
    for steps in (1, 2):
        src = torch.from_numpy(a).cuda()
        dst = torch.full_like(src, float("nan"))
        try:
            plan = b.Plan(dims, R, b.BOX, w, b.PERIODIC, chunk_z=chunk_z or None, **knobs)
        except b.StencilError as e:                    # a tile shape this radius does not have
            assert e.status == b.ERR_UNSUPPORTED and knobs
            return
        with plan as p:
            p.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)
            assert p.query_status() == b.OK
            if dims[-1] % (64 if f64 else 128) == 0:
                assert p.launches == steps
        got = dst.cpu().numpy()
        want = oracle.apply(a, w, b.PERIODIC, steps)
        tol = wl.tolerance(w, float(np.abs(a).max()), steps)
        err = float(np.max(np.abs(got - want)))
        assert err <= tol, f"box R={R} dims={dims} steps={steps} f64={f64}: {err:.3e} > {tol:.3e}"


# ------------------------------------------- periodic boundary under temporal blocking --
@pytest.mark.parametrize("dims,R,knobs", [
    ((21, 37, 256), 1, {}),                                         # one 256-wide region per row, T = 2
    ((33, 50, 128), 1, {}),                                         # 128-wide region
    ((16, 18, 128), 1, dict(fuse_steps=4, tile_x=128)),             # the deepest pass: shells of depth 4
    ((12, 20, 1000), 1, {}),                                        # several regions per row
    ((17, 30, 384), 1, dict(chunk_z=5)),                            # 384-wide region, several z chunks
    ((16, 40, 128), 2, dict(fuse_steps=2, tile_x=128)),             # radius 2: shells of depth 4
    ((4, 4, 128), 1, dict(fuse_steps=2, tile_x=128)),               # the two shells fill the grid in z and y
])
def test_periodic_fused_3d_matches_oracle(dims, R, knobs):
    w = wl.random_star_weights(3, R, 71)
    a = wl.normal_field(dims, 72)
    T = knobs.get("fuse_steps", 0)
    for steps in (2, 3, 5, 9):
        dev = torch.device("cuda:0")
        src = torch.from_numpy(a).to(dev)
        dst = torch.full_like(src, float("nan"))
        with b.Plan(dims, R, b.STAR, w, b.PERIODIC, **knobs) as p:
            depth = p.get(b.KEY_FUSE_STEPS)
            assert depth > 1 and (T == 0 or depth == T)
            p.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)
            assert p.query_status() == b.OK
            passes = -(-steps // depth)
            # a fused pass and its one or two shell kernels; a last single step may wrap inside its sweep
            assert 2 * passes - 1 <= p.launches <= 3 * passes
        got = dst.cpu().numpy()
        want = oracle.apply(a, w, b.PERIODIC, steps)
        tol = wl.tolerance(w, float(np.abs(a).max()), steps)
        err = float(np.max(np.abs(got - want)))
        assert err <= tol, f"dims={dims} R={R} steps={steps}: {err:.3e} > {tol:.3e}"


@pytest.mark.parametrize("R,box,T", [(1, False, 4), (1, True, 4), (2, False, 3), (2, True, 2), (3, False, 2), (4, False, 2)])
@pytest.mark.parametrize("dims", [(67, 132), (200, 260), (16, 16)])
@pytest.mark.parametrize("f64", [False, True])
def test_periodic_fused_2d_matches_oracle(R, box, T, dims, f64):
    if f64 and R > 2:
        pytest.skip("no FP64 cascade beyond radius 2")
    dt = np.float64 if f64 else np.float32
    w = (wl.random_box_weights if box else wl.random_star_weights)(2, R, 73, dt)
    a = wl.normal_field(dims, 74, dt)
    fits = min(dims) >= 2 * T * R
    for steps in (T, T + 1, 2 * T + 1):
        got, used = gpu_sweep(dims, R, b.BOX if box else b.STAR, w, b.PERIODIC, a, steps)
        assert used == "stream"
        want = oracle.apply(a, w, b.PERIODIC, steps)
        tol = wl.tolerance(w, float(np.abs(a).max()), steps)
        err = float(np.max(np.abs(got.astype(np.float64) - want.astype(np.float64))))
        assert err <= tol, f"R={R} box={box} dims={dims} steps={steps} f64={f64} fits={fits}: {err:.3e} > {tol:.3e}"
    with b.Plan(dims, R, b.BOX if box else b.STAR, w, b.PERIODIC) as p:
        assert p.get(b.KEY_FUSE_STEPS) == (T if fits else 1)


def test_periodic_fused_conserves_the_sum_on_a_large_grid():
    """Heat weights sum to 1: under a periodic boundary the total is conserved through fused passes
    (a grid too large for the element-wise oracle)."""
    dims = (256, 256, 256)
    w = wl.star_weights(3, 1, 0.4, [0.1])
    a = wl.uniform_field(dims, 0.0, 1.0, 75)
    src = torch.from_numpy(a).cuda()
    dst = torch.empty_like(src)
    with b.Plan(dims, 1, b.STAR, w, b.PERIODIC) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2
        p.apply(src, dst, 16, torch.cuda.current_stream().cuda_stream)
        assert p.query_status() == b.OK
    total0 = float(src.double().sum())
    total1 = float(dst.double().sum())
    assert abs(total1 - total0) <= 2e-6 * abs(total0)
    assert float(dst.min()) >= 0.0 and float(dst.max()) <= float(src.max())      # max principle
    # the same apply through the unfused wrap-correction route
    ref = torch.empty_like(src)
    with b.Plan(dims, 1, b.STAR, w, b.PERIODIC, fuse_steps=1) as p:
        p.apply(src, ref, 16, torch.cuda.current_stream().cuda_stream)
    assert float((dst - ref).abs().max()) <= 16 * 1e-5 + 1e-6


# ------------------------------------------------- periodic boundary, tiled path --
# periodic_route: None = chosen by the library, 2 = wrap correction after a zero-boundary sweep (extents >= 2R),
# 1 = sweep from a padded copy with wrapped halos
@pytest.mark.parametrize("route", [None, 1, 2])
@pytest.mark.parametrize("R,box", STREAM_OPS)
@pytest.mark.parametrize("dims,chunk_z", [((37, 45, 132), 10), ((8, 16, 128), 0), ((2, 3, 4), 0), ((70, 33, 260), 32),
                                          ((8, 8, 8), 0)])
def test_periodic_3d_on_the_tiled_kernel(R, box, dims, chunk_z, route):
    w = wl.random_box_weights(3, R, 101) if box else wl.random_star_weights(3, R, 101)
    a = wl.normal_field(dims, 102)
    for steps in (1, 2, 3, 6):                       # from 2 steps on the sweeps stay in the padded layout
        used = check(dims, R, b.BOX if box else b.STAR, w, b.PERIODIC, a, steps=steps, chunk_z=chunk_z or None,
                     repeat=2 if steps == 3 else 1, periodic_route=route)
        assert used == "stream"


@pytest.mark.parametrize("route", [None, 1, 2])
@pytest.mark.parametrize("R,box", [(1, False), (4, False), (2, True), (3, True), (4, True)])
@pytest.mark.parametrize("dims", [(67, 132), (3, 8), (200, 260), (8, 8)])
def test_periodic_2d_on_the_tiled_kernel(R, box, dims, route):
    w = wl.random_box_weights(2, R, 103) if box else wl.random_star_weights(2, R, 103)
    a = wl.normal_field(dims, 104)
    for steps in (1, 2, 5):
        used = check(dims, R, b.BOX if box else b.STAR, w, b.PERIODIC, a, steps=steps, repeat=2 if steps == 5 else 1,
                     periodic_route=route)
        assert used == "stream"


def test_periodic_sum_rule_on_gpu():
    """Under a periodic boundary the total is multiplied by sum(w) every step."""
    dims = (48, 40, 64)
    w = wl.star_weights(3, 1, 0.4, [0.1])
    a = wl.uniform_field(dims, 0.0, 1.0, 105)
    got, used = gpu_sweep(dims, 1, b.STAR, w, b.PERIODIC, a, steps=6)
    assert used == "stream"
    s0, s1 = a.astype(np.float64).sum(), got.astype(np.float64).sum()
    assert abs(s1 - s0) < 1e-5 * s0


# ------------------------------------- rows that are not a multiple of 4 floats --
@pytest.mark.parametrize("R,box", [(1, False), (2, False), (3, False), (4, False), (1, True), (2, True)])
@pytest.mark.parametrize("dims", [
    (37, 45, 131),               # two x tiles, the second 3 columns wide; pitch 132
    (9, 20, 6),                  # one padded row holds 6 of 8 floats
    (6, 7, 1),                   # single column
    (40, 30, 257),               # three x tiles, the last one column wide
])
def test_padded_row_sweep_3d(R, box, dims):
    w = wl.random_box_weights(3, R, 51) if box else wl.random_star_weights(3, R, 51)
    a = wl.normal_field(dims, 52)
    used = check(dims, R, b.BOX if box else b.STAR, w, b.ZERO, a)
    assert used == "stream"


@pytest.mark.parametrize("R,box", [(1, False), (4, False), (1, True), (3, True), (4, True)])
@pytest.mark.parametrize("dims", [(67, 133), (200, 259), (5, 3), (33, 1022)])
def test_padded_row_sweep_2d(R, box, dims):
    w = wl.random_box_weights(2, R, 53) if box else wl.random_star_weights(2, R, 53)
    a = wl.normal_field(dims, 54)
    used = check(dims, R, b.BOX if box else b.STAR, w, b.ZERO, a)
    assert used == "stream"


@pytest.mark.parametrize("steps", [0, 1, 2, 3, 6])
@pytest.mark.parametrize("dims", [(21, 40, 137), (90, 201)])
def test_padded_row_iteration(steps, dims):
    """Iterated sweeps stay in the padded layout; what lands in the padding never comes back."""
    ndim = len(dims)
    w = wl.random_box_weights(ndim, 1, 55)
    a = wl.normal_field(dims, 56)
    check(dims, 1, b.BOX, w, b.ZERO, a, steps=steps, repeat=2)
    # same plan, the generic kernel as cross-check of the selection
    used = check(dims, 1, b.BOX, w, b.ZERO, a, steps=steps, variant=b.VARIANT_GENERIC)
    assert used == "generic"


def test_padded_row_host_path_and_scratch_accounting():
    dims = (33, 20, 70)
    w = wl.random_star_weights(3, 2, 57)
    a = wl.normal_field(dims, 58)
    with b.Plan(dims, 2, b.STAR, w, b.ZERO) as p:
        assert p.variant == "stream"
        src = torch.from_numpy(a)
        dst = torch.empty_like(src)
        p.apply_host(src, dst, 3, torch.cuda.current_stream().cuda_stream)
        assert p.query_status() == b.OK
        assert p.get(b.KEY_SCRATCH_BYTES) >= 2 * 33 * 20 * 72 * 4
    got = dst.numpy()
    want = oracle.apply(a, w, b.ZERO, 3)
    assert float(np.max(np.abs(got.astype(np.float64) - want))) <= wl.tolerance(w, float(np.abs(a).max()), 3)


# ------------------------------------------------------------- 2D row streaming --
ROWS2D_OPS = [(1, False), (2, False), (3, False), (4, False), (1, True), (2, True), (3, True), (4, True)]


@pytest.mark.parametrize("R,box", ROWS2D_OPS)
@pytest.mark.parametrize("dims,chunk,stages", [
    ((67, 132), 0, 0),           # two strips, the second 4 columns wide; ragged rows
    ((200, 260), 37, 2),         # several chunks of rows per strip, chunk not a multiple of the batch
    ((3, 8), 0, 0),              # smaller than the stencil reach and than one batch
    ((129, 1024), 16, 4),        # many strips, short chunks
])
def test_rows2d_kernel_matches_oracle(R, box, dims, chunk, stages):
    w = wl.random_box_weights(2, R, 71) if box else wl.random_star_weights(2, R, 71)
    a = wl.normal_field(dims, 72)
    used = check(dims, R, b.BOX if box else b.STAR, w, b.ZERO, a, variant=b.VARIANT_STREAM,
                 chunk_z=chunk or None, stages=stages or None)
    assert used == "stream"


@pytest.mark.parametrize("R,box", [(1, False), (3, True)])
def test_rows2d_iteration(R, box):
    dims = (150, 384)
    w = wl.random_box_weights(2, R, 73) if box else wl.random_star_weights(2, R, 73)
    a = wl.normal_field(dims, 74)
    for steps in (2, 5):
        check(dims, R, b.BOX if box else b.STAR, w, b.ZERO, a, steps=steps)


def test_paper_shaped_2d_box_radius3():
    """The paper's operator (2D box, radius 3, 49 points) on a grid that spans many
    strips and chunks, iterated like its protocol."""
    wk = wl.get("paper2d").scaled((1536, 2048), steps=3)
    a, w = wk.input(), wk.weights()
    got, used = gpu_sweep(wk.dims, wk.radius, wk.shape, w, wk.boundary, a, wk.steps)
    assert used == "stream"
    want = oracle.apply(a, w, wk.boundary, wk.steps)
    assert np.max(np.abs(got - want)) <= wl.tolerance(w, float(np.abs(a).max()), wk.steps)


# ------------------------------------------------------------ 2D temporal blocking --
FUSED2D_OPS = [(1, False, 4), (1, True, 4), (2, False, 3), (2, True, 2), (3, False, 2), (4, False, 2)]   # R, box, T


@pytest.mark.parametrize("R,box,T", FUSED2D_OPS)
@pytest.mark.parametrize("dims,chunk,stages", [
    ((67, 132), 0, 0),           # two strips (each stores 120 columns), ragged in both axes
    ((200, 260), 37, 2),         # three strips, several chunks of rows, chunk not a multiple of the batch
    ((3, 8), 0, 0),              # smaller than the reach of T steps
    ((129, 512), 16, 4),         # five strips; chunks shorter than their halo of T*R rows on either side
    ((300, 120), 0, 0),          # exactly one strip
])
def test_fused_2d_passes_match_oracle(R, box, T, dims, chunk, stages):
    w = wl.random_box_weights(2, R, 71) if box else wl.random_star_weights(2, R, 71)    # sum|w| = 1
    a = wl.normal_field(dims, 72)
    for steps in (T, T + 1, 2 * T + 1, 2):
        dev = torch.device("cuda:0")
        src = torch.from_numpy(a).to(dev)
        dst = torch.full_like(src, float("nan"))
        with b.Plan(dims, R, b.BOX if box else b.STAR, w, b.ZERO, chunk_z=chunk or None, stages=stages or None) as p:
            assert p.variant == "stream" and p.get(b.KEY_FUSE_STEPS) == T
            p.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)
            assert p.query_status() == b.OK
            assert p.launches == -(-steps // T)
        got = dst.cpu().numpy()
        want = oracle.apply(a, w, b.ZERO, steps)
        tol = wl.tolerance(w, float(np.abs(a).max()), steps)
        err = float(np.max(np.abs(got - want)))
        assert err <= tol, f"R={R} box={box} T={T} dims={dims} steps={steps}: {err:.3e} > {tol:.3e}"


def test_fused_2d_equals_unfused_and_keeps_the_zero_boundary():
    dims = (96, 384)
    w = wl.star_weights(2, 1, 0.6, [0.1])                 # heat update: constant fields decay only at the edges
    a = np.ones(dims, dtype=np.float32)
    fused, _ = gpu_sweep(dims, 1, b.STAR, w, b.ZERO, a, steps=8)
    plain, _ = gpu_sweep(dims, 1, b.STAR, w, b.ZERO, a, steps=8, fuse_steps=1)
    want = oracle.apply(a, w, b.ZERO, 8)
    tol = wl.tolerance(w, 1.0, 8)
    assert np.max(np.abs(fused - want)) <= tol and np.max(np.abs(plain - want)) <= tol
    assert fused[0, 0] < 0.5 and abs(fused[48, 192] - 1.0) < 1e-5


@pytest.mark.parametrize("R,box,T", [(1, False, 4), (1, True, 4), (2, False, 3), (2, True, 2)])
@pytest.mark.parametrize("dims,chunk,stages", [
    ((67, 66), 0, 0),            # two strips (each stores 56 columns), ragged in both axes
    ((200, 130), 37, 2),         # three strips, several chunks of rows
    ((3, 8), 0, 0),              # smaller than the reach of T steps
    ((129, 256), 16, 4),         # five strips; chunks shorter than their halo
    ((300, 56), 0, 0),           # exactly one strip
])
def test_f64_fused_2d_passes_match_oracle(R, box, T, dims, chunk, stages):
    mk = wl.random_box_weights if box else wl.random_star_weights
    w = mk(2, R, 73, np.float64)
    a = wl.normal_field(dims, 74, np.float64)
    for steps in (T, T + 1, 2 * T + 1, 2):
        dev = torch.device("cuda:0")
        src = torch.from_numpy(a).to(dev)
        dst = torch.full_like(src, float("nan"))
        with b.Plan(dims, R, b.BOX if box else b.STAR, w, b.ZERO, chunk_z=chunk or None, stages=stages or None) as p:
            assert p.f64 and p.variant == "stream" and p.get(b.KEY_FUSE_STEPS) == T
            p.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)
            assert p.query_status() == b.OK
            assert p.launches == -(-steps // T)
        got = dst.cpu().numpy()
        want = oracle.apply(a, w, b.ZERO, steps)
        tol = wl.tolerance(w, float(np.abs(a).max()), steps)
        err = float(np.max(np.abs(got - want)))
        assert err <= tol, f"R={R} box={box} T={T} dims={dims} steps={steps}: {err:.3e} > {tol:.3e}"


# -------------------------------------------------------------------- fused --
FUSED_CONFIGS = [   # (radius, fuse_steps, region width, region height)
    (1, 2, 256, 32), (1, 2, 256, 16), (1, 3, 256, 32), (1, 4, 128, 32), (1, 2, 128, 32), (1, 3, 128, 32),
    (2, 2, 128, 32), (1, 2, 512, 16), (1, 2, 384, 20),
]


@pytest.mark.parametrize("R,T,width,height", FUSED_CONFIGS)
@pytest.mark.parametrize("dims,chunk_z", [
    ((29, 70, 300), 11),        # several regions in x and y, ragged everywhere, several z chunks
    ((40, 64, 256), 0),         # a 256-wide region spans the whole row (the specialised instantiation)
    ((33, 50, 128), 9),         # the same for the 128-wide regions; ragged in y, several z chunks
    ((21, 37, 512), 8),         # ... and for the 512-wide region, which is loaded as two TMA boxes
    ((19, 30, 452), 0),         # a row that ends inside the second box of a 512-wide region
    ((9, 20, 1000), 0),         # two 512-wide regions per row
    ((17, 41, 384), 6),         # a 384-wide region (three TMA boxes of 128) spans the row
    ((5, 9, 12), 0),            # much smaller than one region
])
def test_fused_passes_match_oracle(R, T, width, height, dims, chunk_z):
    w = wl.random_star_weights(3, R, 61)            # asymmetric taps, sum|w| = 1
    a = wl.normal_field(dims, 62)
    for steps in (T, T + 1, 2 * T + 1):
        dev = torch.device("cuda:0")
        src = torch.from_numpy(a).to(dev)
        dst = torch.full_like(src, float("nan"))
        with b.Plan(dims, R, b.STAR, w, b.ZERO, fuse_steps=T, tile_x=width, fused_tile_y=height,
                    chunk_z=chunk_z or None) as p:
            assert p.get(b.KEY_FUSE_STEPS) == T and p.get(b.KEY_FUSED_TILE_Y) == height
            p.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)
            assert p.query_status() == b.OK
            assert p.launches == -(-steps // T)
        got = dst.cpu().numpy()
        want = oracle.apply(a, w, b.ZERO, steps)
        tol = wl.tolerance(w, float(np.abs(a).max()), steps)
        err = float(np.max(np.abs(got - want)))
        assert err <= tol, f"R={R} T={T} width={width} dims={dims} steps={steps}: {err:.3e} > {tol:.3e}"


FUSED64_CONFIGS = [   # (fuse_steps, region width in doubles): FP64 3D stars of radius 1
    (2, 256), (2, 128), (3, 128),
]


@pytest.mark.parametrize("T,width", FUSED64_CONFIGS)
@pytest.mark.parametrize("dims,chunk_z", [
    ((29, 70, 300), 11),        # several regions in x and y, ragged everywhere, several z chunks
    ((40, 64, 256), 0),         # a 256-wide region spans the whole row (the specialised instantiation)
    ((33, 50, 128), 9),         # the same for the 128-wide regions; ragged in y, several z chunks
    ((19, 30, 230), 0),         # a row that ends inside a 256-wide region
    ((5, 9, 12), 0),            # much smaller than one region
])
def test_f64_fused_3d_passes_match_oracle(T, width, dims, chunk_z):
    """Temporal blocking of FP64 3D grids: the fused kernel with two doubles per lane."""
    w = wl.random_star_weights(3, 1, 61, np.float64)
    a = wl.normal_field(dims, 62, np.float64)
    for steps in (T, T + 1, 2 * T + 1):
        src = torch.from_numpy(a).cuda()
        dst = torch.full_like(src, float("nan"))
        with b.Plan(dims, 1, b.STAR, w, b.ZERO, fuse_steps=T, tile_x=width, chunk_z=chunk_z or None) as p:
            assert p.f64 and p.get(b.KEY_FUSE_STEPS) == T
            p.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)
            assert p.query_status() == b.OK
            assert p.launches == -(-steps // T)
        got = dst.cpu().numpy()
        want = oracle.apply(a, w, b.ZERO, steps)
        tol = wl.tolerance(w, float(np.abs(a).max()), steps)
        err = float(np.max(np.abs(got - want)))
        assert err <= tol, f"T={T} width={width} dims={dims} steps={steps}: {err:.3e} > {tol:.3e}"


@pytest.mark.parametrize("dims", [(20, 452, 128), (12, 450, 480)])
def test_f64_fused_3d_tall_grids_take_32_row_regions(dims):
    """From 448 rows on the 128-wide FP64 regions are 32 rows high by default (one CTA per SM)."""
    w = wl.random_star_weights(3, 1, 63, np.float64)
    a = wl.normal_field(dims, 64, np.float64)
    steps = 5
    src = torch.from_numpy(a).cuda()
    dst = torch.full_like(src, float("nan"))
    with b.Plan(dims, 1, b.STAR, w, b.ZERO) as p:
        assert p.f64 and p.get(b.KEY_FUSE_STEPS) == 2 and p.get(b.KEY_FUSED_TILE_Y) == 32
        p.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)
        assert p.query_status() == b.OK and p.launches == 3
        p.set(b.KEY_FUSED_TILE_Y, 16)
        assert p.get(b.KEY_FUSED_TILE_Y) == 16
    got = dst.cpu().numpy()
    want = oracle.apply(a, w, b.ZERO, steps)
    tol = wl.tolerance(w, float(np.abs(a).max()), steps)
    err = float(np.max(np.abs(got - want)))
    assert err <= tol, f"dims={dims}: {err:.3e} > {tol:.3e}"


def test_f64_fused_3d_is_the_default_where_a_region_spans_the_row():
    """Iterated FP64 applies fuse two steps per pass by default on rows that fill 80 % of the lanes of
    their regions (one region of 128 or 256 doubles, or several 128-wide ones on wider rows); other rows,
    other radii and periodic grids keep one launch per step."""
    w = wl.star_weights(3, 1, 0.4, [0.1]).astype(np.float64)
    for dims, want in [((16, 24, 256), 2), ((16, 24, 128), 2), ((16, 24, 210), 2), ((16, 24, 160), 1),
                       ((16, 24, 512), 2), ((16, 24, 300), 1)]:
        with b.Plan(dims, 1, b.STAR, w, b.ZERO) as p:
            assert p.get(b.KEY_FUSE_STEPS) == want, dims
    with b.Plan((16, 24, 256), 1, b.STAR, w, b.PERIODIC) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1
    with b.Plan((16, 24, 256), 2, b.STAR, wl.random_star_weights(3, 2, 3, np.float64), b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1
    a = wl.uniform_field((16, 24, 256), 0.0, 1.0, 3, np.float64)
    check((16, 24, 256), 1, b.STAR, w, b.ZERO, a, steps=5)
    a = wl.uniform_field((12, 20, 512), 0.0, 1.0, 4, np.float64)
    check((12, 20, 512), 1, b.STAR, w, b.ZERO, a, steps=5)


def test_fused_equals_unfused_within_tolerance_and_keeps_zero_boundary():
    """A field that would leak through the boundary if out-of-grid cells were
    allowed to evolve inside a fused pass: constant ones, heat weights."""
    dims = (20, 30, 64)
    w = wl.star_weights(3, 1, 0.4, [0.1])
    a = np.ones(dims, dtype=np.float32)
    fused, _ = gpu_sweep(dims, 1, b.STAR, w, b.ZERO, a, steps=8, fuse_steps=4, tile_x=128)
    plain, _ = gpu_sweep(dims, 1, b.STAR, w, b.ZERO, a, steps=8, fuse_steps=1)
    want = oracle.apply(a, w, b.ZERO, 8)
    tol = wl.tolerance(w, 1.0, 8)
    assert np.max(np.abs(fused - want)) <= tol and np.max(np.abs(plain - want)) <= tol
    assert fused[0, 0, 0] < 0.5                     # the corner has lost heat to the zero exterior


# ------------------------------------------------------ sharded sweep, one rank --
@pytest.mark.parametrize("halo_steps", [1, 2])
def test_sharded_sweep_single_rank_on_gpu(halo_steps):
    """World size 1 of the slab decomposition runs the real kernels (two steps per round:
    the fused passes) and the result is the plain iterated sweep."""
    from paper_2608_21157_b200.sharded import ShardedSweep
    dims = (40, 48, 128)
    w = wl.star_weights(3, 1, 0.4, [0.1])
    a = wl.uniform_field(dims, 0.0, 1.0, 95)
    sw = ShardedSweep(dims, 1, b.STAR, w, rank=0, world=1, halo_steps=halo_steps)
    try:
        ext = sw.scatter(torch.from_numpy(a).cuda())
        res = sw.apply(ext, 5)
        torch.cuda.synchronize()
        got = sw.interior(res).cpu().numpy()
    finally:
        sw.close()
    want = oracle.apply(a, w, b.ZERO, 5)
    assert np.max(np.abs(got - want)) <= wl.tolerance(w, 1.0, 5)


@pytest.mark.parametrize("boundary", [b.ZERO, b.PERIODIC])
@pytest.mark.parametrize("world,halo_steps,steps", [(2, 1, 3), (3, 2, 5), (4, 2, 4), (2, 3, 6)])
def test_sharded_slabs_with_real_kernels_ranks_emulated_in_one_process(world, halo_steps, steps, boundary):
    """The slabs of 2-4 ranks swept by the real kernels on one GPU, one after the other, with
    the halo exchange done by direct copies between the slabs (no process group, nothing
    waits on anything): ghost depth, edge ranks without outer ghosts and several steps per
    exchange give the sweep of the whole grid.  Under the periodic boundary the ranks form a ring."""
    from paper_2608_21157_b200.sharded import ShardedSweep
    dims = (45, 40, 128)
    R = 1
    w = wl.star_weights(3, R, 0.4, [0.1])
    a = wl.uniform_field(dims, 0.0, 1.0, 96)
    g = torch.from_numpy(a).cuda()
    sws = [ShardedSweep(dims, R, b.STAR, w, boundary, rank=r, world=world, dist=object(), halo_steps=halo_steps)
           for r in range(world)]
    try:
        cur = [sw.scatter(g) for sw in sws]
        other = [torch.empty_like(c) for c in cur]
        D = halo_steps * R
        done = 0
        while done < steps:
            n = min(halo_steps, steps - done)
            own = [sw.interior(c) for sw, c in zip(sws, cur)]
            for r, sw in enumerate(sws):
                assert (sw.lower is None) == (boundary == b.ZERO and r == 0)
                assert (sw.upper is None) == (boundary == b.ZERO and r == world - 1)
                if sw.lower is not None:
                    cur[r][:sw.lo].copy_(own[sw.lower][-D:])
                if sw.upper is not None:
                    cur[r][sw.lo + sw.nlocal:].copy_(own[sw.upper][:D])
            for r, sw in enumerate(sws):
                if sw.overlap:                          # one step per exchange: inner planes, then the edges
                    lo, nl = sw.lo, sw.nlocal
                    inner0 = lo + (R if sw.lower is not None else 0)
                    inner1 = lo + nl - (R if sw.upper is not None else 0)
                    sw._local_apply_planes(cur[r], other[r], inner0, inner1)
                    if inner0 > lo:
                        sw._local_apply_planes(cur[r], other[r], lo, inner0)
                    if inner1 < lo + nl:
                        sw._local_apply_planes(cur[r], other[r], inner1, lo + nl)
                else:
                    sw._local_apply(cur[r], other[r], n)
            cur, other = other, cur
            done += n
        torch.cuda.synchronize()
        got = torch.cat([sw.interior(c) for sw, c in zip(sws, cur)]).cpu().numpy()
    finally:
        for sw in sws:
            sw.close()
    want = oracle.apply(a, w, boundary, steps)
    assert got.shape == want.shape
    assert np.max(np.abs(got - want)) <= wl.tolerance(w, 1.0, steps)


@pytest.mark.parametrize("R,box", [(1, False), (4, False), (1, True), (2, True)])
@pytest.mark.parametrize("dims", [(37, 45, 132), (37, 260)])
@pytest.mark.parametrize("f64", [False, True])
def test_apply_planes_sweeps_exactly_the_requested_planes(R, box, dims, f64):
    """Ranges along the slowest axis: planes of a 3D grid, rows of a 2D grid, fp32 and FP64."""
    nd = len(dims)
    dt = np.float64 if f64 else np.float32
    w = (wl.random_box_weights if box else wl.random_star_weights)(nd, R, 97, dt)
    a = wl.normal_field(dims, 98, dt)
    want = oracle.apply(a, w, b.ZERO, 1)
    tol = wl.tolerance(w, float(np.abs(a).max()), 1)
    src = torch.from_numpy(a).cuda()
    st = torch.cuda.current_stream().cuda_stream
    with b.Plan(dims, R, b.BOX if box else b.STAR, w, b.ZERO) as p:
        assert p.variant == "stream"
        dst = torch.full_like(src, float("nan"))
        p.apply_planes(src, dst, 5, 19, st)
        torch.cuda.synchronize()
        got = dst.cpu().numpy()
        assert np.isnan(got[:5]).all() and np.isnan(got[19:]).all()         # nothing else was written
        assert np.max(np.abs(got[5:19] - want[5:19])) <= tol
        for z0, z1 in ((0, 5), (19, 36), (36, 37)):                          # the rest, in three more ranges
            p.apply_planes(src, dst, z0, z1, st)
        torch.cuda.synchronize()
        assert p.query_status() == b.OK
        assert np.max(np.abs(dst.cpu().numpy() - want)) <= tol
        for z0, z1 in ((-1, 4), (3, 38), (7, 7), (9, 2)):
            with pytest.raises(b.StencilError) as e:
                p.apply_planes(src, dst, z0, z1, st)
            assert e.value.status == b.ERR_INVALID
    with b.Plan(dims, R, b.BOX if box else b.STAR, w, b.PERIODIC) as p:
        with pytest.raises(b.StencilError) as e:
            p.apply_planes(src, torch.empty_like(src), 0, 4, st)
        assert e.value.status == b.ERR_UNSUPPORTED
    with b.Plan(dims, R, b.BOX if box else b.STAR, w, b.ZERO, variant=b.VARIANT_GENERIC) as p:
        with pytest.raises(b.StencilError) as e:
            p.apply_planes(src, torch.empty_like(src), 0, 4, st)
        assert e.value.status == b.ERR_UNSUPPORTED
    if f64:                                             # the fp32 entry point refuses an FP64 plan and vice versa
        with b.Plan(dims, R, b.BOX if box else b.STAR, w, b.ZERO) as p:
            assert b.stencil_apply_planes(p._h, src.data_ptr(), dst.data_ptr(), 0, 4, st) == b.ERR_INVALID


@pytest.mark.parametrize("dims,f64", [((45, 260), False), ((45, 40, 64), True), ((45, 130), True)])
def test_sharded_overlap_on_2d_and_fp64_slabs(dims, f64):
    """The exchange/compute overlap of the slab decomposition (ranged sweeps) beyond 3D fp32: the slabs of
    three emulated ranks, one step per exchange, exchange by direct copies."""
    from paper_2608_21157_b200.sharded import ShardedSweep
    world, steps, R = 3, 3, 1
    dt = np.float64 if f64 else np.float32
    w = wl.random_star_weights(len(dims), R, 101, dt)
    a = wl.normal_field(dims, 102, dt)
    g = torch.from_numpy(a).cuda()
    sws = [ShardedSweep(dims, R, b.STAR, w, rank=r, world=world, dist=object()) for r in range(world)]
    try:
        assert all(sw.overlap for sw in sws)
        cur = [sw.scatter(g) for sw in sws]
        other = [torch.empty_like(c) for c in cur]
        for _ in range(steps):
            own = [sw.interior(c) for sw, c in zip(sws, cur)]
            for r, sw in enumerate(sws):
                if sw.lower is not None:
                    cur[r][:sw.lo].copy_(own[sw.lower][-R:])
                if sw.upper is not None:
                    cur[r][sw.lo + sw.nlocal:].copy_(own[sw.upper][:R])
            for r, sw in enumerate(sws):
                lo, nl = sw.lo, sw.nlocal
                inner0 = lo + (R if sw.lower is not None else 0)
                inner1 = lo + nl - (R if sw.upper is not None else 0)
                sw._local_apply_planes(cur[r], other[r], inner0, inner1)
                if inner0 > lo:
                    sw._local_apply_planes(cur[r], other[r], lo, inner0)
                if inner1 < lo + nl:
                    sw._local_apply_planes(cur[r], other[r], inner1, lo + nl)
            cur, other = other, cur
        torch.cuda.synchronize()
        got = torch.cat([sw.interior(c) for sw, c in zip(sws, cur)]).cpu().numpy()
    finally:
        for sw in sws:
            sw.close()
    want = oracle.apply(a, w, b.ZERO, steps)
    assert np.max(np.abs(got - want)) <= wl.tolerance(w, float(np.abs(a).max()), steps)


# --------------------------------------------------------------------- FP64 --
def check_f64(dims, R, shape, w, boundary, a, steps=1, **kw):
    assert a.dtype == np.float64 and w.dtype == np.float64
    got, used = gpu_sweep(dims, R, shape, w, boundary, a, steps, **kw)
    assert got.dtype == np.float64
    want = oracle.apply(a, w, boundary, steps)
    tol = wl.tolerance(w, float(np.abs(a).max()), steps)
    err = float(np.max(np.abs(got - want)))
    assert err <= tol, f"{used}: max err {err:.3e} > tol {tol:.3e} for dims={dims} R={R} steps={steps}"
    return used


@pytest.mark.parametrize("R,box", [(1, False), (2, False), (3, False), (4, False), (1, True), (2, True), (3, True),
                                   (4, True)])
@pytest.mark.parametrize("dims,chunk,stages", [
    ((67, 66), 0, 0),            # two 64-column strips, the second 2 columns wide
    ((200, 258), 37, 2),         # several chunks of rows, chunk not a multiple of the batch
    ((3, 8), 0, 0),              # smaller than the stencil reach
    ((129, 512), 16, 4),
])
def test_f64_rows2d_kernel_matches_oracle(R, box, dims, chunk, stages):
    mk = wl.random_box_weights if box else wl.random_star_weights
    w = mk(2, R, 81, np.float64)
    a = wl.normal_field(dims, 82, np.float64)
    used = check_f64(dims, R, b.BOX if box else b.STAR, w, b.ZERO, a, chunk_z=chunk or None, stages=stages or None)
    assert used == "stream"


@pytest.mark.parametrize("R,box", [(1, False), (2, False), (3, False), (4, False), (1, True), (2, True)])
@pytest.mark.parametrize("dims,chunk_z,stages", [
    ((37, 45, 66), 10, 3),       # two 64-column tiles, ragged in x, y and z
    ((8, 16, 64), 0, 0),         # exactly one tile
    ((3, 5, 4), 0, 2),           # smaller than the stencil reach
    ((70, 33, 130), 32, 0),      # three x tiles, the last 2 points wide
])
def test_f64_stream_kernel_matches_oracle(R, box, dims, chunk_z, stages):
    w = (wl.random_box_weights if box else wl.random_star_weights)(3, R, 85, np.float64)
    a = wl.normal_field(dims, 86, np.float64)
    for steps in (1, 3):
        used = check_f64(dims, R, b.BOX if box else b.STAR, w, b.ZERO, a, steps=steps,
                         chunk_z=chunk_z or None, stages=stages or None)
        assert used == "stream"


@pytest.mark.parametrize("dims,R,box,boundary", [
    ((33, 47), 3, True, b.ZERO), ((20, 30), 2, True, b.PERIODIC), ((9, 12, 21), 1, True, b.ZERO),
    ((7, 10, 14), 2, False, b.PERIODIC), ((40, 64), 5, True, b.ZERO), ((9, 12, 20), 2, True, b.ZERO)])
def test_f64_generic_kernel(dims, R, box, boundary):
    ndim = len(dims)
    w = (wl.random_box_weights if box else wl.random_star_weights)(ndim, R, 83, np.float64)
    a = wl.normal_field(dims, 84, np.float64)
    used = check_f64(dims, R, b.BOX if box else b.STAR, w, boundary, a, steps=3, variant=b.VARIANT_GENERIC)
    assert used == "generic"


@pytest.mark.parametrize("dims,R,box", [
    ((33, 47), 3, True), ((200, 259), 1, False), ((5, 1), 2, True), ((129, 513), 4, False),
    ((9, 12, 21), 1, True), ((37, 45, 67), 4, False), ((70, 33, 131), 2, False), ((6, 7, 1), 1, False)])
@pytest.mark.parametrize("steps", [1, 4])
def test_f64_padded_row_sweep(dims, R, box, steps):
    """Rows of an odd number of doubles run on the tiled kernels between grids with padded rows."""
    ndim = len(dims)
    w = (wl.random_box_weights if box else wl.random_star_weights)(ndim, R, 87, np.float64)
    a = wl.normal_field(dims, 88, np.float64)
    used = check_f64(dims, R, b.BOX if box else b.STAR, w, b.ZERO, a, steps=steps, repeat=2)
    assert used == "stream"


@pytest.mark.parametrize("dims,R,box", [
    ((37, 45, 66), 1, False), ((37, 45, 66), 4, False), ((8, 16, 64), 1, True), ((2, 3, 2), 2, False),
    ((70, 33, 130), 3, False),
    ((67, 66), 3, True), ((3, 8), 4, False), ((200, 258), 1, False), ((64, 2), 2, True)])
@pytest.mark.parametrize("route", [None, 1, 2])
def test_f64_periodic_on_the_tiled_kernels(dims, R, box, route):
    ndim = len(dims)
    w = (wl.random_box_weights if box else wl.random_star_weights)(ndim, R, 89, np.float64)
    a = wl.normal_field(dims, 90, np.float64)
    for steps in (1, 2, 5):
        used = check_f64(dims, R, b.BOX if box else b.STAR, w, b.PERIODIC, a, steps=steps, periodic_route=route)
        assert used == "stream"


def test_f64_paper_shaped_box_iterated_and_type_checks():
    """The paper's operator in its own precision: 2D box radius 3, FP64, iterated."""
    wk = wl.get("paper2d_f64").scaled((768, 1024), steps=3)
    a, w = wk.input(), wk.weights()
    assert check_f64(wk.dims, wk.radius, wk.shape, w, wk.boundary, a, wk.steps) == "stream"
    # a plan only serves the apply call of its own precision
    src = torch.zeros(64, 64, dtype=torch.float64, device="cuda")
    dst = torch.zeros_like(src)
    with b.Plan((64, 64), 3, b.BOX, wl.random_box_weights(2, 3, 1, np.float64), b.ZERO) as p:
        assert b.stencil_apply(p._h, src.data_ptr(), dst.data_ptr(), 1, 0) == b.ERR_INVALID
        assert b.stencil_apply_host(p._h, src.data_ptr(), dst.data_ptr(), 1, 0) == b.ERR_INVALID
    with b.Plan((64, 64), 3, b.BOX, wl.random_box_weights(2, 3, 1), b.ZERO) as p:
        assert b.stencil_apply_f64(p._h, src.data_ptr(), dst.data_ptr(), 1, 0) == b.ERR_INVALID


# ------------------------------------------------------------ bounded waits --
# (family, dims, radius, box, FP64, boundary, time steps, plan knobs, launches of the family's kernel per apply)
_WAIT_CASES = [
    ("stream", (8, 16, 128), 1, False, False, b.ZERO, 1, {}, 1),
    ("stream box", (8, 16, 128), 1, True, False, b.ZERO, 1, {}, 1),
    ("stream wrap", (8, 16, 128), 1, False, False, b.PERIODIC, 1, {}, 1),
    ("fused 3d", (8, 16, 128), 1, False, False, b.ZERO, 2, {"fuse_steps": 2}, 1),
    ("rows2d", (24, 128), 1, False, False, b.ZERO, 1, {}, 1),
    ("rows2d box", (24, 128), 3, True, False, b.ZERO, 1, {}, 1),
    ("rows2d fused", (40, 128), 1, False, False, b.ZERO, 4, {}, 1),
    ("stream f64", (8, 16, 64), 1, False, True, b.ZERO, 1, {}, 1),
    ("stream f64 wrap", (8, 16, 64), 1, False, True, b.PERIODIC, 1, {}, 1),
    ("rows2d f64", (24, 64), 2, False, True, b.ZERO, 1, {}, 1),
    ("rows2d fused f64", (40, 64), 1, False, True, b.ZERO, 4, {}, 1),
]


@pytest.mark.parametrize("family,dims,R,box,f64,boundary,steps,knobs,launches", _WAIT_CASES,
                         ids=[c[0].replace(" ", "_") for c in _WAIT_CASES])
def test_expired_device_wait_is_reported_and_the_context_stays_usable(family, dims, R, box, f64, boundary, steps,
                                                                      knobs, launches):
    """Failure detection without a fault, for every family of tiled kernels: the thread that
    requests the input is told never to load one plane (3D) or batch of rows (2D), so the
    bounded wait for it runs out (64 polls of at most 20 us), the kernel returns early, and the
    host reads STENCIL_ERR_TIMEOUT from the status word.  Nothing traps or spins forever; the
    next apply on the same plan is correct again."""
    dt = np.float64 if f64 else np.float32
    ndim = len(dims)
    if steps > 1:                                    # iterated: non-negative weights that sum to one
        w = wl.star_weights(ndim, 1, 1.0 - 0.2 * ndim, [0.1]).astype(dt)
    else:
        w = (wl.random_box_weights if box else wl.random_star_weights)(ndim, R, 5, dt)
    a = wl.uniform_field(dims, -1.0, 1.0, 91, dt)
    src = torch.from_numpy(a).cuda()
    dst = torch.zeros_like(src)
    stream = torch.cuda.current_stream().cuda_stream
    with b.Plan(dims, R, b.BOX if box else b.STAR, w, boundary, variant=b.VARIANT_STREAM, **knobs) as p:
        p.set(b.KEY_WAIT_POLLS, 64)
        p.set(b.KEY_TEST_DROP_PLANE, 0)
        l0 = p.launches
        p.apply(src, dst, steps, stream)
        assert p.launches - l0 == launches, f"{family}: the apply did not take the route under test"
        assert p.query_status() == b.ERR_TIMEOUT
        assert p.query_status() == b.OK              # the word is cleared by the query
        p.set(b.KEY_TEST_DROP_PLANE, -1)
        p.set(b.KEY_WAIT_POLLS, 1 << 20)
        p.apply(src, dst, steps, stream)
        assert p.query_status() == b.OK
    torch.cuda.synchronize()
    want = oracle.apply(a, w, boundary, steps)
    err = np.max(np.abs(dst.cpu().numpy().astype(np.float64) - want.astype(np.float64)))
    assert err <= wl.tolerance(w, 1.0, steps)        # the bound follows the dtype of the weights


# ----------------------------------------------------- the five full configs --
@pytest.mark.parametrize("name", wl.BASELINE_CONFIGS)
def test_baseline_config_full_size(name):
    """Full-size grids, default plan (the launch configuration the benchmark
    times), every point compared with the oracle."""
    wk = wl.get(name)
    a = wk.input()
    w = wk.weights()
    got, used = gpu_sweep(wk.dims, wk.radius, wk.shape, w, wk.boundary, a, wk.steps)
    want = oracle.apply(a, w, wk.boundary, wk.steps)
    tol = wl.tolerance(w, float(np.abs(a).max()), wk.steps)
    err = float(np.max(np.abs(got - want)))
    assert err <= tol, f"{name} ({used}): max err {err:.3e} > tol {tol:.3e}"
    if name == "cfg5":
        # max principle of the heat update: 0 <= u <= max u0
        assert got.min() >= 0.0 and got.max() <= a.max()


@pytest.mark.parametrize("boundary", [b.ZERO, b.PERIODIC])
def test_default_fused_passes_of_a_tall_256_wide_grid(boundary):
    """From 448 rows on a 256-wide grid takes 256 x 32 regions by default (one CTA per SM): an odd number
    of steps, so that a single step follows the fused passes, against the oracle."""
    dims, R, steps = (24, 452, 256), 1, 5
    w = wl.random_star_weights(3, R, 321)
    a = wl.normal_field(dims, 322)
    with b.Plan(dims, R, b.STAR, w, boundary) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2 and p.get(b.KEY_FUSED_TILE_Y) == 32
    got, used = gpu_sweep(dims, R, b.STAR, w, boundary, a, steps)
    want = oracle.apply(a, w, boundary, steps)
    tol = wl.tolerance(w, float(np.abs(a).max()), steps)
    err = float(np.max(np.abs(got - want)))
    assert err <= tol, f"{used}: max err {err:.3e} > tol {tol:.3e}"


@pytest.mark.parametrize("boundary", [b.ZERO, b.PERIODIC])
def test_fused_passes_whose_last_planes_go_to_short_chunks(boundary):
    """256 x 512 x 512, two steps per pass in 43 regions of 512 x 16, one CTA per SM: three equal chunks
    per region would occupy 129 of a B200's 148 SMs, so the launcher cuts the last planes of every region
    into shorter chunks whose CTAs come last in the grid.  Every point of two passes against the oracle;
    the output starts as NaN, so a plane that no chunk covers shows."""
    dims, R, steps = (256, 512, 512), 1, 4
    w = wl.random_star_weights(3, R, 311)
    a = wl.normal_field(dims, 312)
    got, used = gpu_sweep(dims, R, b.STAR, w, boundary, a, steps)
    want = oracle.apply(a, w, boundary, steps)
    tol = wl.tolerance(w, float(np.abs(a).max()), steps)
    err = float(np.max(np.abs(got - want)))
    assert err <= tol, f"{used}: max err {err:.3e} > tol {tol:.3e}"


def test_paper_workload_full_grid_one_step():
    """The paper's grid at full size (10240 x 10240, 49-point box), one time step, every
    point against the oracle, in the launch configuration the benchmark times."""
    wk = wl.get("paper2d")
    a, w = wk.input(), wk.weights()
    got, used = gpu_sweep(wk.dims, wk.radius, wk.shape, w, wk.boundary, a, 1)
    assert used == "stream"
    want = oracle.apply(a, w, wk.boundary, 1)
    assert float(np.max(np.abs(got - want))) <= wl.tolerance(w, float(np.abs(a).max()), 1)


def test_grid_with_more_than_2_to_the_31_points():
    """Maximum-size case: 2100 x 1024 x 1024 = 2.2e9 points (8.8 GB per grid), beyond 32-bit
    element offsets.  The field is a formula of the indices, built on the device; sampled
    output planes (first, middle, last) are compared with the oracle run on the 2R+1 input
    planes around them, built from the same formula on the host."""
    nz, ny, nx = 2100, 1024, 1024
    R = 1
    w = wl.random_star_weights(3, R, 97)

    def field(z_lo, z_hi, xp):
        z = xp.arange(z_lo, z_hi).reshape(-1, 1, 1)
        y = xp.arange(ny).reshape(1, -1, 1)
        x = xp.arange(nx).reshape(1, 1, -1)
        return (((x * 3 + y * 5 + z * 7) % 17) - 8)

    dev = torch.device("cuda:0")
    src = torch.empty((nz, ny, nx), dtype=torch.float32, device=dev)
    for z0 in range(0, nz, 100):
        z1 = min(z0 + 100, nz)
        src[z0:z1] = field(z0, z1, torch).to(dev).float() / 8.0
    dst = torch.empty_like(src)
    with b.Plan((nz, ny, nx), R, b.STAR, w, b.ZERO) as p:
        assert p.variant == "stream"
        p.apply(src, dst, 1, torch.cuda.current_stream().cuda_stream)
        assert p.query_status() == b.OK
    torch.cuda.synchronize()
    tol = wl.tolerance(w, 1.0, 1)
    for zc in (0, 1049, nz - 1):
        lo, hi = max(zc - R, 0), min(zc + R + 1, nz)
        # planes outside the grid are zero: pad so that the oracle's own boundary is never the answer
        sub = np.zeros((2 * R + 1, ny, nx), dtype=np.float32)
        sub[lo - (zc - R):hi - (zc - R)] = (field(lo, hi, np) / 8.0).astype(np.float32)
        want = oracle.apply(sub, w, b.ZERO, 1)[R]
        got = dst[zc].cpu().numpy()
        assert float(np.max(np.abs(got - want))) <= tol, f"plane {zc}"
    del src, dst
    torch.cuda.empty_cache()


def test_periodic_fused_pass_on_a_grid_with_more_than_2_to_the_31_points():
    """The same grid under the periodic boundary, two steps in one fused pass (three 384-wide regions
    per row) plus the two shell kernels: sampled output planes, among them the wrapped ones at both
    ends, against the oracle run on the 5 input planes around each (the centre plane of such a block
    does not depend on how the block ends in z)."""
    nz, ny, nx = 2100, 1024, 1024
    R, steps = 1, 2
    w = wl.random_star_weights(3, R, 103)

    def field(zs, xp):
        z = zs.reshape(-1, 1, 1)
        y = xp.arange(ny).reshape(1, -1, 1)
        x = xp.arange(nx).reshape(1, 1, -1)
        return (((x * 3 + y * 5 + z * 7) % 17) - 8)

    dev = torch.device("cuda:0")
    src = torch.empty((nz, ny, nx), dtype=torch.float32, device=dev)
    for z0 in range(0, nz, 100):
        z1 = min(z0 + 100, nz)
        src[z0:z1] = field(torch.arange(z0, z1), torch).to(dev).float() / 8.0
    dst = torch.empty_like(src)
    with b.Plan((nz, ny, nx), R, b.STAR, w, b.PERIODIC) as p:
        assert p.variant == "stream" and p.get(b.KEY_FUSE_STEPS) == 2
        p.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)
        assert p.query_status() == b.OK
        assert p.launches == 3
    torch.cuda.synchronize()
    tol = wl.tolerance(w, 1.0, steps)
    H = steps * R
    for zc in (0, 1, 1049, nz - 2, nz - 1):
        zs = np.arange(zc - H, zc + H + 1) % nz
        sub = (field(zs, np) / 8.0).astype(np.float32)
        want = oracle.apply(sub, w, b.PERIODIC, steps)[H]
        got = dst[zc].cpu().numpy()
        assert float(np.max(np.abs(got - want))) <= tol, f"plane {zc}"
    del src, dst
    torch.cuda.empty_cache()


def test_2d_grid_with_more_than_2_to_the_31_points():
    """The same for the 2D row-streaming kernel: 46400 x 46400 = 2.15e9 points."""
    ny = nx = 46400
    R = 2
    w = wl.random_box_weights(2, R, 98)

    def field(y_lo, y_hi, xp):
        y = xp.arange(y_lo, y_hi).reshape(-1, 1)
        x = xp.arange(nx).reshape(1, -1)
        return (((x * 3 + y * 5) % 17) - 8)

    dev = torch.device("cuda:0")
    src = torch.empty((ny, nx), dtype=torch.float32, device=dev)
    for y0 in range(0, ny, 4000):
        y1 = min(y0 + 4000, ny)
        src[y0:y1] = field(y0, y1, torch).to(dev).float() / 8.0
    dst = torch.empty_like(src)
    with b.Plan((ny, nx), R, b.BOX, w, b.ZERO) as p:
        assert p.variant == "stream"
        p.apply(src, dst, 1, torch.cuda.current_stream().cuda_stream)
        assert p.query_status() == b.OK
    torch.cuda.synchronize()
    tol = wl.tolerance(w, 1.0, 1)
    for yc in (0, 23111, ny - 1):
        lo, hi = max(yc - R, 0), min(yc + R + 1, ny)
        sub = np.zeros((2 * R + 1, nx), dtype=np.float32)
        sub[lo - (yc - R):hi - (yc - R)] = (field(lo, hi, np) / 8.0).astype(np.float32)
        want = oracle.apply(sub, w, b.ZERO, 1)[R]
        got = dst[yc].cpu().numpy()
        assert float(np.max(np.abs(got - want))) <= tol, f"row {yc}"
    # two time steps in one fused pass on the same grid; the band of rows around a sampled row ends
    # either at the grid's own edge or 2R rows away from the row, so the row itself is exact
    with b.Plan((ny, nx), R, b.BOX, w, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2
        p.apply(src, dst, 2, torch.cuda.current_stream().cuda_stream)
        assert p.query_status() == b.OK and p.launches == 1
    torch.cuda.synchronize()
    tol = wl.tolerance(w, 1.0, 2)
    for yc in (0, 3, 23111, ny - 1):
        lo, hi = max(yc - 2 * R, 0), min(yc + 2 * R + 1, ny)
        band = (field(lo, hi, np) / 8.0).astype(np.float32)
        want = oracle.apply(band, w, b.ZERO, 2)[yc - lo]
        got = dst[yc].cpu().numpy()
        assert float(np.max(np.abs(got - want))) <= tol, f"row {yc}, two fused steps"
    del src, dst
    torch.cuda.empty_cache()


def test_generic_kernel_on_a_full_3d_config():
    wk = wl.get("cfg2").scaled((128, 128, 128))
    a, w = wk.input(), wk.weights()
    check(wk.dims, wk.radius, wk.shape, w, wk.boundary, a, variant=b.VARIANT_GENERIC)


# ------------------------------------------------- non-finite input at a face --
@pytest.mark.parametrize("variant", [b.VARIANT_GENERIC, b.VARIANT_STREAM], ids=["generic", "stream"])
@pytest.mark.parametrize("dims", [(24, 128), (6, 10, 128)], ids=["2d", "3d"])
def test_infinity_at_a_face_does_not_leak_through_taps_that_leave_the_grid(dims, variant):
    """A tap that leaves the grid contributes an exact zero whatever the grid holds next to the face.
    With one +Inf at a corner point and a star whose taps are all non-zero, the result is infinite
    exactly where a tap reaches the corner and finite (no NaN) everywhere else, on both kernel
    families: the one-thread-per-point kernel once loaded the thread's own point for such a tap and
    multiplied it by a zero weight, which turned the corner itself into NaN."""
    ndim = len(dims)
    a = wl.uniform_field(dims, -1.0, 1.0, 17)
    a[(0,) * ndim] = np.inf
    w = wl.random_star_weights(ndim, 1, 3)
    assert np.count_nonzero(w) == 1 + 2 * ndim
    got, used = gpu_sweep(dims, 1, b.STAR, w, b.ZERO, a, 1, variant=variant)
    want = oracle.apply(a, w, b.ZERO, 1)
    assert not np.isnan(want).any()
    inf = np.isinf(want)
    assert np.array_equal(np.isinf(got), inf) and np.array_equal(np.sign(got[inf]), np.sign(want[inf]))
    assert np.max(np.abs(got[~inf] - want[~inf])) <= wl.tolerance(w, 1.0, 1)
