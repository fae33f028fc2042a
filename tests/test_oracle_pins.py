"""Pins of the CPU oracle against things other than itself.

The oracle evaluates out[p] = sum_o w[o] * in[p+o] (zero-padded or periodic
cross-correlation, stride 1; the paper's case-study protocol), iterated with
one float32 rounding per step.  Each test below fixes part of that against a
closed form, an invariant, brute force, or an independent library routine, so
that a dropped tap, a sign, a flipped kernel, a transposed axis, a wrong
boundary rule or a wrong rounding point fails at least one of them.
"""
import json
import os

import numpy as np
import pytest

import oracle
from paper_2608_21157_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
ZERO, PERIODIC = oracle.ZERO, oracle.PERIODIC


def rand_weights(ndim, R, seed, star=False):
    return wl.random_star_weights(ndim, R, seed) if star else wl.random_box_weights(ndim, R, seed)


# ---------------------------------------------------------------- golden --
@pytest.mark.parametrize("name", ["laplace5_3x3", "shift_dx_plus1_3x3", "shift_dz_minus1_2x2x2"])
def test_hand_worked_examples(name):
    with open(os.path.join(GOLDEN, name + ".json")) as f:
        g = json.load(f)
    w = np.array(g["weights"], dtype=np.float32)
    a = np.array(g["in"], dtype=np.float32)
    want = np.array(g["out"], dtype=np.float32)
    got = oracle.apply(a, w, ZERO, g["steps"])
    assert np.array_equal(got, want)


# ------------------------------------------------------- 1 constant field --
@pytest.mark.parametrize("dims,R", [((9, 11), 1), ((8, 9), 3), ((6, 7, 9), 1), ((10, 9, 11), 2)])
def test_constant_field_all_ones_box_zero_boundary(dims, R):
    """All-ones box on a constant field c: out[p] = c * prod_axes (#in-range taps)."""
    ndim = len(dims)
    w = np.ones((2 * R + 1,) * ndim, dtype=np.float32)
    c = 3.0
    a = np.full(dims, c, dtype=np.float32)
    got = oracle.apply(a, w, ZERO, 1)
    want = np.full(dims, c, dtype=np.float64)
    for ax, n in enumerate(dims):
        idx = np.arange(n)
        cnt = np.minimum(idx + R, n - 1) - np.maximum(idx - R, 0) + 1
        shape = [1] * ndim
        shape[ax] = n
        want = want * cnt.reshape(shape)
    assert np.array_equal(got, want.astype(np.float32))


@pytest.mark.parametrize("ndim,R", [(2, 1), (2, 3), (3, 1), (3, 2)])
def test_constant_field_periodic_gives_sum_w(ndim, R):
    rng = np.random.default_rng(10 + ndim + R)
    w = rng.integers(-4, 5, size=(2 * R + 1,) * ndim).astype(np.float32)  # exact arithmetic
    dims = (7, 6, 9)[:ndim] if ndim == 3 else (7, 9)
    a = np.full(dims, 5.0, dtype=np.float32)
    got = oracle.apply(a, w, PERIODIC, 1)
    assert np.array_equal(got, np.full(dims, 5.0 * w.astype(np.float64).sum(), dtype=np.float32))


def test_constant_field_interior_gives_sum_w_zero_boundary():
    w = wl.star_weights(3, 1, -6.0, [1.0])
    a = np.full((8, 8, 8), 2.0, dtype=np.float32)
    got = oracle.apply(a, w, ZERO, 1)
    assert np.all(got[1:-1, 1:-1, 1:-1] == 0.0)
    assert got[0, 0, 0] == 2.0 * (-6 + 3)      # three neighbours inside
    assert got[0, 3, 3] == 2.0 * (-6 + 5)      # face point: five neighbours inside


# ------------------------------------------------------ 2 quadratic field --
def test_laplacian_of_quadratic_2d_and_3d_is_exact():
    ny, nx = 16, 18
    y, x = np.meshgrid(np.arange(ny), np.arange(nx), indexing="ij")
    f = (3 * x * x + 2 * y * y + 5 * x - 7 * y + 11).astype(np.float32)
    got = oracle.apply(f, wl.star_weights(2, 1, -4.0, [1.0]), ZERO, 1)
    assert np.all(got[1:-1, 1:-1] == 2 * (3 + 2))

    nz = 12
    z, y, x = np.meshgrid(np.arange(nz), np.arange(ny), np.arange(nx), indexing="ij")
    f = (3 * x * x + 2 * y * y - 4 * z * z + x - y + 2 * z + 1).astype(np.float32)
    got = oracle.apply(f, wl.star_weights(3, 1, -6.0, [1.0]), ZERO, 1)
    assert np.all(got[1:-1, 1:-1, 1:-1] == 2 * (3 + 2 - 4))


def test_fd8_laplacian_moments_and_quadratic():
    """The radius-4 coefficients annihilate constants and degree 4/6/8 terms and
    give second moment 2 per axis; on a quadratic the interior value is 2(a+b+c)."""
    c = [float(wl.FD8_CENTER_1D)] + [float(v) for v in wl.FD8_AXIS]
    k = np.arange(1, 5, dtype=np.float64)
    ax = np.array(c[1:])
    assert abs(c[0] + 2 * ax.sum()) < 1e-14
    assert abs(2 * (ax * k ** 2).sum() - 2.0) < 1e-13
    for p in (4, 6, 8):
        assert abs(2 * (ax * k ** p).sum()) < 1e-9
    n = 20
    z, y, x = np.meshgrid(np.arange(n), np.arange(n), np.arange(n), indexing="ij")
    f = (2 * x * x + 3 * y * y + 1 * z * z + x + 2 * y - z + 4).astype(np.float32)
    got = oracle.apply(f, wl.fd8_laplacian_weights(3), ZERO, 1)
    inner = got[4:-4, 4:-4, 4:-4].astype(np.float64)
    # rational weights are rounded to float32: |error| <= 2^-24 * sum|w| * max|f|
    bound = 2.0 ** -23 * 19.6 * float(f.max())
    assert np.max(np.abs(inner - 2 * (2 + 3 + 1))) < bound


# ------------------------------------------------------------- 3 impulse --
@pytest.mark.parametrize("ndim,R,boundary", [(2, 1, ZERO), (2, 3, ZERO), (3, 1, ZERO), (3, 2, PERIODIC), (2, 2, PERIODIC)])
def test_impulse_response_is_the_point_reflected_weights(ndim, R, boundary):
    w = rand_weights(ndim, R, 21)
    dims = (4 * R + 3, 4 * R + 2, 4 * R + 5)[:ndim]
    p0 = tuple(d // 2 for d in dims)
    a = np.zeros(dims, dtype=np.float32)
    a[p0] = 1.0
    got = oracle.apply(a, w, boundary, 1)
    want = np.zeros(dims, dtype=np.float32)
    for o in np.ndindex(*w.shape):
        off = tuple(int(i) - R for i in o)
        q = tuple(p0[k] - off[k] for k in range(ndim))     # out[p0 - o] = w[o]
        want[q] = w[o]
    assert np.array_equal(got, want)


def test_impulse_near_corner_zero_boundary_drops_outside_taps():
    R = 2
    w = rand_weights(2, R, 22)
    a = np.zeros((6, 7), dtype=np.float32)
    a[0, 1] = 1.0
    got = oracle.apply(a, w, ZERO, 1)
    for y in range(6):
        for x in range(7):
            oy, ox = 0 - y, 1 - x      # p + o = p0
            inside = abs(oy) <= R and abs(ox) <= R
            assert got[y, x] == (w[oy + R, ox + R] if inside else 0.0)


# --------------------------------------------------- 4 periodic sum rule --
@pytest.mark.parametrize("ndim,R", [(2, 2), (3, 1), (3, 3)])
def test_periodic_sum_rule(ndim, R):
    w = rand_weights(ndim, R, 31)
    dims = (9, 10, 12)[:ndim]
    a = wl.normal_field(dims, 32)
    got = oracle.apply(a, w, PERIODIC, 1).astype(np.float64).sum()
    want = w.astype(np.float64).sum() * a.astype(np.float64).sum()
    assert abs(got - want) <= 1e-6 * np.abs(a).astype(np.float64).sum() * np.abs(w).sum()


def test_symmetric_unit_sum_stencil_conserves_total_under_periodic():
    w = wl.star_weights(3, 1, 0.4, [0.1])
    a = wl.uniform_field((12, 10, 14), 0.0, 1.0, 33)
    out = oracle.apply(a, w, PERIODIC, 5)
    s0, s1 = a.astype(np.float64).sum(), out.astype(np.float64).sum()
    assert abs(s1 - s0) < 1e-5 * s0


# ------------------------------------------------ 5 periodic Fourier mode --
def test_periodic_fourier_symbol_fd8():
    n = 32
    k = (1, 2, 3)
    z, y, x = np.meshgrid(np.arange(n), np.arange(n), np.arange(n), indexing="ij")
    phase = 2 * np.pi * (k[0] * z + k[1] * y + k[2] * x) / n
    f = np.cos(phase).astype(np.float32)
    w = wl.fd8_laplacian_weights(3)
    got = oracle.apply(f, w, PERIODIC, 1).astype(np.float64)
    # symbol of a symmetric star: centre + sum_axis sum_j 2 c_j cos(2 pi k_axis j / n)
    wd = w.astype(np.float64)
    lam = wd[4, 4, 4]
    for ax in range(3):
        for j in range(1, 5):
            idx = [4, 4, 4]
            idx[ax] += j
            lam += 2 * wd[tuple(idx)] * np.cos(2 * np.pi * k[ax] * j / n)
    assert np.max(np.abs(got - lam * f.astype(np.float64))) < 5e-6
    # and the symbol approximates -|kappa|^2 to eighth order
    kap2 = sum((2 * np.pi * kk / n) ** 2 for kk in k)
    assert abs(lam + kap2) < 2e-4 * kap2


# -------------------------------- 6 sine eigenmodes, zero boundary, steps --
@pytest.mark.parametrize("steps", [1, 7, 64])
def test_heat_sine_eigenmode_decay_zero_boundary(steps):
    dims = (32, 30, 28)
    m = (1, 2, 3)
    c, a_nb = np.float32(0.4), np.float32(0.1)
    w = wl.star_weights(3, 1, float(c), [float(a_nb)])
    u = np.ones(dims, dtype=np.float64)
    mu = float(c)
    for ax, n in enumerate(dims):
        shape = [1, 1, 1]
        shape[ax] = n
        u = u * np.sin(np.pi * m[ax] * (np.arange(n) + 1) / (n + 1)).reshape(shape)
        mu += 2 * float(a_nb) * np.cos(np.pi * m[ax] / (n + 1))
    u0 = u.astype(np.float32)
    got = oracle.apply(u0, w, ZERO, steps).astype(np.float64)
    want = (mu ** steps) * u0.astype(np.float64)
    assert np.max(np.abs(got - want)) < 2e-7 * steps + 1e-7


def test_sine_eigenmode_2d_laplacian():
    dims = (17, 23)
    m = (2, 5)
    w = wl.star_weights(2, 1, -4.0, [1.0])
    u = np.ones(dims)
    mu = -4.0
    for ax, n in enumerate(dims):
        shape = [1, 1]
        shape[ax] = n
        u = u * np.sin(np.pi * m[ax] * (np.arange(n) + 1) / (n + 1)).reshape(shape)
        mu += 2 * np.cos(np.pi * m[ax] / (n + 1))
    u0 = u.astype(np.float32)
    got = oracle.apply(u0, w, ZERO, 1).astype(np.float64)
    assert np.max(np.abs(got - mu * u0)) < 1e-6


# ------------------------------------------- 7 brute force dense matrix --
def _dense_operator(dims, w, boundary):
    """N x N matrix built by SCATTER: column q feeds row p = q - o with w[o]."""
    ndim = len(dims)
    R = (w.shape[0] - 1) // 2
    N = int(np.prod(dims))
    A = np.zeros((N, N), dtype=np.float64)
    strides = [int(np.prod(dims[k + 1:])) for k in range(ndim)]
    for q in np.ndindex(*dims):
        col = sum(q[k] * strides[k] for k in range(ndim))
        for o in np.ndindex(*w.shape):
            off = [int(i) - R for i in o]
            p = [q[k] - off[k] for k in range(ndim)]
            if boundary == PERIODIC:
                # every p with (p + o) mod n == q; for n <= R several images can coincide
                p = [pp % dims[k] for k, pp in enumerate(p)]
            elif any(pp < 0 or pp >= dims[k] for k, pp in enumerate(p)):
                continue
            row = sum(p[k] * strides[k] for k in range(ndim))
            A[row, col] += float(w[o])
    return A


@pytest.mark.parametrize("dims,R,star,boundary", [
    ((5, 7), 1, False, ZERO), ((5, 7), 2, False, PERIODIC), ((6, 5), 3, True, ZERO),
    ((2, 3), 3, False, ZERO), ((2, 3), 2, False, PERIODIC), ((1, 9), 1, False, ZERO),
    ((3, 4, 5), 1, False, ZERO), ((3, 4, 5), 1, False, PERIODIC), ((4, 3, 6), 2, True, ZERO),
    ((2, 2, 7), 2, False, PERIODIC), ((1, 1, 5), 1, False, ZERO), ((5, 4, 3), 2, False, ZERO),
])
def test_brute_force_dense_matrix(dims, R, star, boundary):
    ndim = len(dims)
    w = rand_weights(ndim, R, 41 + R, star=star)
    a = wl.normal_field(dims, 42)
    A = _dense_operator(dims, w, boundary)
    want = (A @ a.astype(np.float64).ravel()).reshape(dims)
    got = oracle.apply(a, w, boundary, 1)
    # summation order differs -> compare in double before the cast, then after
    assert np.max(np.abs(got.astype(np.float64) - want)) < 1e-6
    assert np.array_equal(got, want.astype(np.float32)) or \
        np.max(np.abs(got - want.astype(np.float32))) <= np.spacing(np.float32(np.abs(want).max()))


def test_brute_force_iterated():
    dims, R = (4, 5, 3), 1
    w = rand_weights(3, R, 43)
    a = wl.normal_field(dims, 44)
    A = _dense_operator(dims, w, ZERO)
    v = a.astype(np.float64).ravel()
    for _ in range(5):
        v = (A @ v).astype(np.float32).astype(np.float64)   # one fp32 rounding per step
    got = oracle.apply(a, w, ZERO, 5)
    assert np.max(np.abs(got.astype(np.float64).ravel() - v)) < 1e-7


# ----------------------------------------------- 8 library special cases --
@pytest.mark.parametrize("dims,R,star", [((33, 47), 3, False), ((40, 31), 1, True),
                                         ((19, 23, 29), 1, False), ((24, 20, 27), 4, True),
                                         ((13, 17, 19), 2, False)])
def test_matches_torch_conv_float64_zero_padding(dims, R, star):
    import torch
    import torch.nn.functional as F
    ndim = len(dims)
    w = rand_weights(ndim, R, 51, star=star)
    a = wl.normal_field(dims, 52)
    conv = F.conv2d if ndim == 2 else F.conv3d
    want = conv(torch.from_numpy(a).double()[None, None], torch.from_numpy(w).double()[None, None],
                padding=R)[0, 0].numpy()
    got = oracle.apply(a, w, ZERO, 1)
    assert np.max(np.abs(got.astype(np.float64) - want)) < 2e-7
    assert np.max(np.abs(got - want.astype(np.float32))) <= np.spacing(np.float32(np.abs(want).max()))


@pytest.mark.parametrize("dims,R,boundary,mode", [
    ((21, 34), 3, ZERO, "constant"), ((21, 34), 2, PERIODIC, "wrap"),
    ((11, 14, 17), 1, ZERO, "constant"), ((11, 14, 17), 2, PERIODIC, "wrap")])
def test_matches_scipy_correlate(dims, R, boundary, mode):
    from scipy import ndimage
    w = rand_weights(len(dims), R, 53)
    a = wl.normal_field(dims, 54)
    want = ndimage.correlate(a.astype(np.float64), w.astype(np.float64), mode=mode, cval=0.0)
    got = oracle.apply(a, w, boundary, 1)
    assert np.max(np.abs(got.astype(np.float64) - want)) < 2e-7


# ------------------------------------------------- 9 linearity and shift --
def test_linearity_and_periodic_shift_equivariance():
    dims = (9, 8, 10)
    w = rand_weights(3, 2, 61)
    a, b = wl.normal_field(dims, 62), wl.normal_field(dims, 63)
    sa, sb = oracle.apply(a, w, ZERO, 1), oracle.apply(b, w, ZERO, 1)
    comb = oracle.apply((2 * a - 3 * b).astype(np.float32), w, ZERO, 1)
    assert np.max(np.abs(comb - (2 * sa - 3 * sb))) < 2e-5
    shifted = np.roll(a, (2, -3, 1), axis=(0, 1, 2))
    assert np.array_equal(oracle.apply(shifted, w, PERIODIC, 1),
                          np.roll(oracle.apply(a, w, PERIODIC, 1), (2, -3, 1), axis=(0, 1, 2)))


# ------------------------------------------------------ 10 time stepping --
@pytest.mark.parametrize("boundary", [ZERO, PERIODIC])
def test_time_composition_is_bit_identical(boundary):
    dims = (8, 9, 7)
    w = wl.star_weights(3, 1, 0.4, [0.1])
    a = wl.uniform_field(dims, 0.0, 1.0, 71)
    once = oracle.apply(a, w, boundary, 7)
    twice = oracle.apply(oracle.apply(a, w, boundary, 3), w, boundary, 4)
    assert np.array_equal(once, twice)
    assert np.array_equal(oracle.apply(a, w, boundary, 0), a)
    assert not np.shares_memory(oracle.apply(a, w, boundary, 0), a)


def test_rounding_happens_once_per_step():
    """An intermediate that needs more than 24 bits: 1 + 2^-24 rounds to 1 in
    float32.  Two steps with per-step rounding lose the small term; a double
    carried across steps would keep it."""
    w = np.zeros((3, 3), dtype=np.float32)
    w[1, 1] = 1.0
    w[1, 2] = np.float32(2.0 ** -24)
    a = np.zeros((1, 3), dtype=np.float32)
    a[0, 0] = 1.0
    a[0, 1] = 1.0
    one = oracle.apply(a, w, ZERO, 1)
    assert one[0, 0] == np.float32(1.0)            # 1 + 2^-24 ties to even -> 1
    w2 = w.copy()
    w2[1, 2] = np.float32(2.0 ** -23)
    assert oracle.apply(a, w2, ZERO, 1)[0, 0] == np.float32(1.0 + 2.0 ** -23)


# ----------------------------------------------------- 11 max principle --
def test_max_principle_and_heat_loss_zero_boundary():
    w = wl.star_weights(3, 1, 0.4, [0.1])
    a = wl.uniform_field((20, 18, 22), 0.0, 1.0, 81)
    prev_sum = a.astype(np.float64).sum()
    u = a
    for _ in range(6):
        u = oracle.apply(u, w, ZERO, 1)
        assert u.min() >= 0.0 and u.max() <= a.max()
        s = u.astype(np.float64).sum()
        assert s <= prev_sum
        prev_sum = s


# --------------------------------------------------------- spot-check API --
def test_points_entry_matches_full_sweep():
    dims = (9, 13, 11)
    w = rand_weights(3, 2, 91)
    a = wl.normal_field(dims, 92)
    full = oracle.apply(a, w, ZERO, 1).ravel()
    idx = np.random.default_rng(93).integers(0, a.size, size=200)
    assert np.array_equal(oracle.apply_points(a, w, idx, ZERO), full[idx])
    fullp = oracle.apply(a, w, PERIODIC, 1).ravel()
    assert np.array_equal(oracle.apply_points(a, w, idx, PERIODIC), fullp[idx])


def test_grids_smaller_than_the_stencil():
    w = np.ones((7, 7), dtype=np.float32)
    a = np.arange(6, dtype=np.float32).reshape(2, 3)
    assert np.all(oracle.apply(a, w, ZERO, 1) == a.sum())
    # periodic with n < 2R+1: each cell is hit several times by the wrapped taps
    cnt_y = [sum(1 for d in range(-3, 4) if (y + d) % 2 == yy) for y in [0] for yy in range(2)]
    cnt_x = [sum(1 for d in range(-3, 4) if (0 + d) % 3 == xx) for xx in range(3)]
    want = sum(a[yy, xx] * cnt_y[yy] * cnt_x[xx] for yy in range(2) for xx in range(3))
    assert oracle.apply(a, w, PERIODIC, 1)[0, 0] == want


# ------------------------------------------------ FP64 entry point (long double sums) --
@pytest.mark.parametrize("name", ["laplace5_3x3", "shift_dx_plus1_3x3", "shift_dz_minus1_2x2x2"])
def test_f64_hand_worked_examples(name):
    with open(os.path.join(GOLDEN, name + ".json")) as f:
        g = json.load(f)
    got = oracle.apply(np.array(g["in"], dtype=np.float64), np.array(g["weights"], dtype=np.float64), ZERO, 1)
    assert got.dtype == np.float64
    assert np.array_equal(got, np.array(g["out"], dtype=np.float64))


@pytest.mark.parametrize("ndim,R,boundary", [(2, 3, ZERO), (3, 1, ZERO), (3, 2, PERIODIC)])
def test_f64_impulse_response(ndim, R, boundary):
    w = wl.random_box_weights(ndim, R, 21, np.float64)
    dims = (4 * R + 3, 4 * R + 2, 4 * R + 5)[:ndim]
    p0 = tuple(d // 2 for d in dims)
    a = np.zeros(dims)
    a[p0] = 1.0
    got = oracle.apply(a, w, boundary, 1)
    want = np.zeros(dims)
    for o in np.ndindex(*w.shape):
        want[tuple(p0[k] - (int(o[k]) - R) for k in range(ndim))] = w[o]
    assert np.array_equal(got, want)


@pytest.mark.parametrize("dims,R,star,boundary", [
    ((5, 7), 3, False, ZERO), ((6, 5), 2, False, PERIODIC), ((2, 3), 3, False, ZERO),
    ((3, 4, 5), 1, False, ZERO), ((4, 3, 6), 2, True, PERIODIC)])
def test_f64_brute_force_dense_matrix(dims, R, star, boundary):
    ndim = len(dims)
    w = (wl.random_star_weights if star else wl.random_box_weights)(ndim, R, 41 + R, np.float64)
    a = wl.normal_field(dims, 42, np.float64)
    A = _dense_operator(dims, w, boundary).astype(np.longdouble)
    want = (A @ a.astype(np.longdouble).ravel()).reshape(dims)
    got = oracle.apply(a, w, boundary, 1)
    # long double sums in another order: after the cast to double at most one unit in the last place apart
    assert np.max(np.abs(got - want.astype(np.float64))) <= np.spacing(np.abs(want).max().astype(np.float64))


@pytest.mark.parametrize("dims,R", [((33, 47), 3), ((13, 17, 19), 2)])
def test_f64_matches_torch_conv_and_scipy(dims, R):
    import torch
    import torch.nn.functional as F
    from scipy import ndimage
    ndim = len(dims)
    w = wl.random_box_weights(ndim, R, 51, np.float64)
    a = wl.normal_field(dims, 52, np.float64)
    conv = F.conv2d if ndim == 2 else F.conv3d
    want = conv(torch.from_numpy(a)[None, None], torch.from_numpy(w)[None, None], padding=R)[0, 0].numpy()
    got = oracle.apply(a, w, ZERO, 1)
    # the library sums in double: its own rounding error bounds the distance
    bound = (2 * R + 1) ** ndim * 2.0 ** -52 * np.abs(w).sum() * np.abs(a).max()
    assert np.max(np.abs(got - want)) <= bound
    wrap = ndimage.correlate(a, w, mode="wrap")
    assert np.max(np.abs(oracle.apply(a, w, PERIODIC, 1) - wrap)) <= bound


def test_f64_laplacian_quadratic_composition_and_rounding_point():
    ny, nx = 16, 18
    y, x = np.meshgrid(np.arange(ny), np.arange(nx), indexing="ij")
    f = (3 * x * x + 2 * y * y + 5 * x - 7 * y + 11).astype(np.float64)
    got = oracle.apply(f, wl.star_weights(2, 1, -4.0, [1.0]).astype(np.float64), ZERO, 1)
    assert np.all(got[1:-1, 1:-1] == 10.0)
    w = wl.random_box_weights(2, 3, 5, np.float64)
    a = wl.uniform_field((20, 24), -1.0, 1.0, 6, np.float64)
    assert np.array_equal(oracle.apply(a, w, ZERO, 5), oracle.apply(oracle.apply(a, w, ZERO, 2), w, ZERO, 3))
    # 1 + 2^-53 is a tie in double and rounds to 1; the long double sum must round once, at the end
    w2 = np.zeros((3, 3)); w2[1, 1] = 1.0; w2[1, 2] = 2.0 ** -53
    b2 = np.zeros((1, 3)); b2[0, 0] = 1.0; b2[0, 1] = 1.0
    assert oracle.apply(b2, w2, ZERO, 1)[0, 0] == 1.0
    w2[1, 2] = 2.0 ** -52
    assert oracle.apply(b2, w2, ZERO, 1)[0, 0] == 1.0 + 2.0 ** -52
    # and it really carries more than double inside: (1 + 2^-53) + 2^-53 = 1 + 2^-52 exactly
    w3 = np.zeros((3, 3)); w3[1, 0] = 2.0 ** -53; w3[1, 1] = 1.0; w3[1, 2] = 2.0 ** -53
    b3 = np.ones((1, 3))
    assert oracle.apply(b3, w3, ZERO, 1)[0, 1] == 1.0 + 2.0 ** -52
