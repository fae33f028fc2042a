"""Seeded synthetic workloads for the stencil sweep.

This module only *describes* problems: grid sizes, the dense weight array of
each stencil and the seeded input field.  It contains none of the sweep's
arithmetic and imports neither the CUDA binding nor the CPU oracle, so both
sides can be fed the very same host arrays.

Conventions (shared by every consumer):

* ``dims`` is slowest axis first, ``(nz, ny, nx)`` or ``(ny, nx)``; x is
  contiguous.
* ``weights`` is the dense cross-correlation kernel of shape ``(2R+1,)*ndim``
  in the same axis order; entry ``[dz+R, dy+R, dx+R]`` multiplies
  ``in[p + (dz, dy, dx)]``.  A star stencil is a dense array whose off-axis
  entries are exactly zero.
* Random numbers come from ``numpy.random.default_rng(seed)``, drawn in
  float64 in C order and cast to float32 once.

The paper's case study (Case-study protocol, RQ3) measures a 2D box stencil of
radius 3 on a 10240 x 10240 grid; it publishes no weights and no data, so the
workloads here are synthetic stand-ins with the same shapes and structure.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field
from fractions import Fraction
from typing import Callable, Dict, Tuple

import numpy as np

STAR = 0
BOX = 1
ZERO = 0
PERIODIC = 1


# --------------------------------------------------------------------------
# dense weight arrays
# --------------------------------------------------------------------------
def star_weights(ndim: int, radius: int, center: float, axis_coeffs) -> np.ndarray:
    """Dense (2R+1)^ndim array with ``center`` in the middle and
    ``axis_coeffs[k-1]`` at distance k along every axis (both directions)."""
    R = radius
    w = np.zeros((2 * R + 1,) * ndim, dtype=np.float64)
    mid = (R,) * ndim
    w[mid] = center
    for ax in range(ndim):
        for k in range(1, R + 1):
            for sgn in (-1, 1):
                idx = list(mid)
                idx[ax] += sgn * k
                w[tuple(idx)] = axis_coeffs[k - 1]
    return w.astype(np.float32)


def random_box_weights(ndim: int, radius: int, seed: int, dtype=np.float32) -> np.ndarray:
    """(2R+1)^ndim weights uniform[-1,1) in dense C order, scaled so that the
    absolute values sum to one (in float64), then cast to ``dtype``."""
    rng = np.random.default_rng(seed)
    w = rng.uniform(-1.0, 1.0, size=(2 * radius + 1,) * ndim)
    w = w / np.abs(w).sum()
    return w.astype(dtype)


def random_star_weights(ndim: int, radius: int, seed: int, dtype=np.float32) -> np.ndarray:
    """Asymmetric star: every on-axis tap gets its own uniform[-1,1) value."""
    rng = np.random.default_rng(seed)
    R = radius
    w = np.zeros((2 * R + 1,) * ndim, dtype=np.float64)
    mid = (R,) * ndim
    w[mid] = rng.uniform(-1.0, 1.0)
    for ax in range(ndim):
        for k in range(-R, R + 1):
            if k == 0:
                continue
            idx = list(mid)
            idx[ax] += k
            w[tuple(idx)] = rng.uniform(-1.0, 1.0)
    w = w / np.abs(w).sum()
    return w.astype(dtype)


#: per-axis coefficients of the 8th-order central second difference
#: (distance 1..4) and its centre value, as exact rationals.
FD8_AXIS = (Fraction(8, 5), Fraction(-1, 5), Fraction(8, 315), Fraction(-1, 560))
FD8_CENTER_1D = Fraction(-205, 72)


def fd8_laplacian_weights(ndim: int = 3) -> np.ndarray:
    """25-point (3D) star of radius 4: centre ndim * (-205/72), per axis
    8/5, -1/5, 8/315, -1/560; each rational rounded once to float32."""
    center = float(FD8_CENTER_1D * ndim)
    return star_weights(ndim, 4, center, [float(c) for c in FD8_AXIS])


# --------------------------------------------------------------------------
# input fields
# --------------------------------------------------------------------------
def uniform_field(dims, lo: float, hi: float, seed: int, dtype=np.float32) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.uniform(lo, hi, size=tuple(dims)).astype(dtype)


def normal_field(dims, seed: int, dtype=np.float32) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.standard_normal(size=tuple(dims)).astype(dtype)


def smooth_sine_field(dims, seed: int, noise: float = 1e-3) -> np.ndarray:
    """prod_axis sin(2 pi idx / n_axis) + noise * N(0,1), built in float64 on
    integer indices (one period across each axis), cast once to float32."""
    dims = tuple(int(d) for d in dims)
    f = np.ones(dims, dtype=np.float64)
    for ax, n in enumerate(dims):
        shape = [1] * len(dims)
        shape[ax] = n
        f = f * np.sin(2.0 * np.pi * np.arange(n, dtype=np.float64) / n).reshape(shape)
    rng = np.random.default_rng(seed)
    f = f + noise * rng.standard_normal(size=dims)
    return f.astype(np.float32)


# --------------------------------------------------------------------------
# workload table
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    description: str
    dims: Tuple[int, ...]
    radius: int
    shape: int
    boundary: int
    steps: int
    make_weights: Callable[[], np.ndarray] = field(repr=False)
    make_input: Callable[[], np.ndarray] = field(repr=False)
    dtype: type = np.float32          # float32, or float64 (the paper's own precision)

    @property
    def itemsize(self) -> int:
        return int(np.dtype(self.dtype).itemsize)

    @property
    def ndim(self) -> int:
        return len(self.dims)

    @property
    def npoints(self) -> int:
        n = 1
        for d in self.dims:
            n *= int(d)
        return n

    @property
    def point_updates(self) -> int:
        return self.npoints * max(self.steps, 1)

    def weights(self) -> np.ndarray:
        w = np.ascontiguousarray(self.make_weights(), dtype=self.dtype)
        assert w.shape == (2 * self.radius + 1,) * self.ndim
        return w

    def input(self) -> np.ndarray:
        a = np.ascontiguousarray(self.make_input(), dtype=self.dtype)
        assert a.shape == tuple(self.dims)
        return a

    def taps(self) -> int:
        return int(np.count_nonzero(self.weights()))

    def scaled(self, dims, steps=None, name=None) -> "Workload":
        """Same operator and input recipe on another grid size (for parity
        cases the oracle finishes quickly and for bounded CPU samples)."""
        dims = tuple(int(d) for d in dims)
        old_make = self.make_input
        # the input recipes below close over dims via _with_dims
        maker = getattr(old_make, "_with_dims", None)
        if maker is None:
            raise ValueError("workload input recipe is not resizable")
        return Workload(
            name=name or f"{self.name}@{'x'.join(map(str, dims))}",
            description=self.description,
            dims=dims,
            radius=self.radius,
            shape=self.shape,
            boundary=self.boundary,
            steps=self.steps if steps is None else int(steps),
            make_weights=self.make_weights,
            make_input=maker(dims),
            dtype=self.dtype,
        )


def _resizable(fn: Callable[[Tuple[int, ...]], np.ndarray], dims):
    """Bind ``dims`` into an input recipe but keep it re-bindable."""
    def make():
        return fn(tuple(dims))
    make._with_dims = lambda d: _resizable(fn, d)  # type: ignore[attr-defined]
    return make


def _build_table() -> Dict[str, Workload]:
    t: Dict[str, Workload] = {}

    t["cfg1"] = Workload(
        "cfg1", "2D 5-point Laplacian 256x256, zero boundary, 1 step",
        (256, 256), 1, STAR, ZERO, 1,
        lambda: star_weights(2, 1, -4.0, [1.0]),
        _resizable(lambda d: uniform_field(d, -1.0, 1.0, 0), (256, 256)))

    t["cfg2"] = Workload(
        "cfg2", "3D 7-point star R=1 512^3 (centre -6, neighbours +1, h=1), zero boundary, 1 step",
        (512, 512, 512), 1, STAR, ZERO, 1,
        lambda: star_weights(3, 1, -6.0, [1.0]),
        _resizable(lambda d: uniform_field(d, -1.0, 1.0, 1), (512, 512, 512)))

    t["cfg3"] = Workload(
        "cfg3", "3D 27-point box R=1 512^3, random weights with sum|w|=1, zero boundary, 1 step",
        (512, 512, 512), 1, BOX, ZERO, 1,
        lambda: random_box_weights(3, 1, 2),
        _resizable(lambda d: normal_field(d, 3), (512, 512, 512)))

    t["cfg4"] = Workload(
        "cfg4", "3D 25-point star R=4 (8th-order FD Laplacian) 512^3, zero boundary, 1 step",
        (512, 512, 512), 4, STAR, ZERO, 1,
        lambda: fd8_laplacian_weights(3),
        _resizable(lambda d: smooth_sine_field(d, 4), (512, 512, 512)))

    t["cfg5"] = Workload(
        "cfg5", "3D 7-point heat diffusion u += 0.1*(sum nb - 6u), 256^3, 64 steps, zero boundary",
        (256, 256, 256), 1, STAR, ZERO, 64,
        lambda: star_weights(3, 1, 1.0 - 6 * 0.1, [0.1]),
        _resizable(lambda d: uniform_field(d, 0.0, 1.0, 5), (256, 256, 256)))

    # supplementary: the paper's own shape (2D box radius 3, 49 points,
    # 10240^2), in fp32 with seeded weights since the paper prints none.
    t["paper2d"] = Workload(
        "paper2d", "2D 49-point box R=3 10240^2, random weights sum|w|=1, zero boundary, 16 steps",
        (10240, 10240), 3, BOX, ZERO, 16,
        lambda: random_box_weights(2, 3, 7),
        _resizable(lambda d: uniform_field(d, -1.0, 1.0, 6), (10240, 10240)))

    # the same in the paper's own precision: FP64 fields and weights (800 MiB per grid)
    t["paper2d_f64"] = Workload(
        "paper2d_f64", "2D 49-point box R=3 10240^2 in FP64, random weights sum|w|=1, zero boundary, 16 steps",
        (10240, 10240), 3, BOX, ZERO, 16,
        lambda: random_box_weights(2, 3, 7, np.float64),
        _resizable(lambda d: uniform_field(d, -1.0, 1.0, 6, np.float64), (10240, 10240)),
        dtype=np.float64)

    # supplementary: cfg2's operator with a periodic boundary
    t["cfg2_periodic"] = Workload(
        "cfg2_periodic", "3D 7-point star R=1 512^3, periodic boundary, 1 step",
        (512, 512, 512), 1, STAR, PERIODIC, 1,
        lambda: star_weights(3, 1, -6.0, [1.0]),
        _resizable(lambda d: uniform_field(d, -1.0, 1.0, 1), (512, 512, 512)))

    # supplementary: the iterated 2D heat update (5 points) on the paper's grid size
    t["heat2d"] = Workload(
        "heat2d", "2D 5-point heat update u += 0.1*(sum nb - 4u), 10240^2, 16 steps, zero boundary",
        (10240, 10240), 1, STAR, ZERO, 16,
        lambda: star_weights(2, 1, 1.0 - 4 * 0.1, [0.1]),
        _resizable(lambda d: uniform_field(d, 0.0, 1.0, 10), (10240, 10240)))

    # supplementary: the widest box the tiled 3D kernel covers (125 taps: bound by the FMA pipe)
    t["box3d_r2"] = Workload(
        "box3d_r2", "3D 125-point box R=2 512^3, random weights with sum|w|=1, zero boundary, 1 step",
        (512, 512, 512), 2, BOX, ZERO, 1,
        lambda: random_box_weights(3, 2, 8),
        _resizable(lambda d: normal_field(d, 9), (512, 512, 512)))

    # supplementary: the iterated heat update on a periodic 512^3 grid (stable weights)
    t["cfg5L_periodic"] = Workload(
        "cfg5L_periodic", "3D 7-point heat update R=1 512^3, periodic boundary, 16 steps",
        (512, 512, 512), 1, STAR, PERIODIC, 16,
        lambda: star_weights(3, 1, 0.4, [0.1]),
        _resizable(lambda d: uniform_field(d, 0.0, 1.0, 5), (512, 512, 512)))

    # supplementary: two of the 3D configs in FP64 (1 GiB per grid)
    t["cfg2_f64"] = Workload(
        "cfg2_f64", "3D 7-point star R=1 512^3 in FP64 (centre -6, neighbours +1), zero boundary, 1 step",
        (512, 512, 512), 1, STAR, ZERO, 1,
        lambda: star_weights(3, 1, -6.0, [1.0]).astype(np.float64),
        _resizable(lambda d: uniform_field(d, -1.0, 1.0, 1, np.float64), (512, 512, 512)),
        dtype=np.float64)
    t["cfg4_f64"] = Workload(
        "cfg4_f64", "3D 25-point star R=4 512^3 in FP64 (8th-order FD Laplacian), zero boundary, 1 step",
        (512, 512, 512), 4, STAR, ZERO, 1,
        lambda: star_weights(3, 4, float(FD8_CENTER_1D * 3), [float(c) for c in FD8_AXIS]).astype(np.float64),
        _resizable(lambda d: uniform_field(d, -1.0, 1.0, 4, np.float64), (512, 512, 512)),
        dtype=np.float64)

    # supplementary: the iterated heat update in FP64 (1 GiB per grid) and an iterated 27-point box
    t["cfg5L_f64"] = Workload(
        "cfg5L_f64", "3D 7-point heat diffusion 512^3 in FP64, 16 steps, zero boundary",
        (512, 512, 512), 1, STAR, ZERO, 16,
        lambda: star_weights(3, 1, 1.0 - 6 * 0.1, [0.1]).astype(np.float64),
        _resizable(lambda d: uniform_field(d, 0.0, 1.0, 5, np.float64), (512, 512, 512)),
        dtype=np.float64)
    t["box27_iterated"] = Workload(
        "box27_iterated", "3D 27-point box R=1 512^3, random weights with sum|w|=1, zero boundary, 16 steps",
        (512, 512, 512), 1, BOX, ZERO, 16,
        lambda: random_box_weights(3, 1, 2),
        _resizable(lambda d: normal_field(d, 3), (512, 512, 512)))

    # supplementary: the iterated heat operator on a grid that does not fit L2
    t["cfg5L"] = Workload(
        "cfg5L", "3D 7-point heat diffusion 512^3, 16 steps (working set exceeds L2)",
        (512, 512, 512), 1, STAR, ZERO, 16,
        lambda: star_weights(3, 1, 1.0 - 6 * 0.1, [0.1]),
        _resizable(lambda d: uniform_field(d, 0.0, 1.0, 5), (512, 512, 512)))
    return t


WORKLOADS: Dict[str, Workload] = _build_table()
BASELINE_CONFIGS = ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5")


def get(name: str) -> Workload:
    return WORKLOADS[name]


def sha256(a: np.ndarray) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def tolerance(weights: np.ndarray, max_abs_in: float, steps: int) -> float:
    """Acceptance bound max|gpu - oracle| <= 1e-5 * sum|w| * max|in| * steps + 1e-6
    (sum in float64 over the float32 weights; steps counted as at least 1).

    For float64 weights (FP64 sweeps) the same form with the constants scaled by the ratio of
    the unit roundoffs, 2^-53 / 2^-24: 2e-14 * sum|w| * max|in| * steps + 2e-15.  A K-term
    FMA chain errs by at most about K * 2^-53 * sum|w| * max|in| (5.4e-15 relative for the
    49-point box), which leaves the same margin as the float32 bound does."""
    sw = float(np.abs(weights.astype(np.float64)).sum())
    if weights.dtype == np.float64:
        return 2e-14 * sw * float(max_abs_in) * max(int(steps), 1) + 2e-15
    return 1e-5 * sw * float(max_abs_in) * max(int(steps), 1) + 1e-6
