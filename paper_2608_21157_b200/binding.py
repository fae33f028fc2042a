"""ctypes binding of the C ABI in ``include/stencil.h``.

Argument marshalling only: every sweep runs in the CUDA kernels of
``libstencil_b200.so``.  There is no CPU fallback; if the library has not been
built, loading raises.  Device memory and streams come from the caller
(PyTorch in the tests and the benchmark).

With ``STENCIL_B200_DEBUG=1`` in the environment the binding loads the debug
build, ``libstencil_b200_debug.so`` (``python -m paper_2608_21157_b200.build
--debug``), whose kernels check every store against the output grid.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
DEBUG_BUILD = os.environ.get("STENCIL_B200_DEBUG", "0") == "1"
LIB_PATH = os.path.join(_HERE, "libstencil_b200_debug.so" if DEBUG_BUILD else "libstencil_b200.so")

STAR, BOX = 0, 1
ZERO, PERIODIC = 0, 1

OK, ERR_INVALID, ERR_UNSUPPORTED, ERR_CUDA, ERR_ALLOC, ERR_TIMEOUT, ERR_TOO_LARGE, ERR_BOUNDS = 0, -1, -2, -3, -4, -5, -6, -7
STATIC_MAX_POINTS = 1 << 21

VARIANT_AUTO, VARIANT_GENERIC, VARIANT_STREAM, VARIANT_FUSED = 0, 1, 2, 3

(KEY_VARIANT, KEY_TILE_X, KEY_TILE_Y, KEY_FUSE_STEPS, KEY_LAUNCHES, KEY_SCRATCH_BYTES,
 KEY_CHUNK_Z, KEY_STAGES, KEY_STREAMING_STORE, KEY_ROWS_PER_THREAD, KEY_WAIT_POLLS,
 KEY_TEST_DROP_PLANE, KEY_CHAIN_LAUNCHES, KEY_FUSED_TILE_Y, KEY_PERIODIC_ROUTE, KEY_DEVICE,
 KEY_DEBUG_SHRINK) = range(17)

#: every symbol include/stencil.h declares
EXPORTS = (
    "stencil_plan", "stencil_apply", "stencil_plan_f64", "stencil_apply_f64",
    "stencil_apply_host", "stencil_apply_static", "stencil_apply_planes", "stencil_apply_planes_f64",
    "stencil_destroy",
    "stencil_status_string", "stencil_variant_name", "stencil_query_status",
    "stencil_plan_set", "stencil_plan_get",
)

_lib = None


class StencilError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def load() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2608_21157_b200.build"
            f"{' --debug' if DEBUG_BUILD else ''}` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64p, f32p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_float)
    lib.stencil_plan.restype = ctypes.c_int
    lib.stencil_plan.argtypes = [ctypes.POINTER(vp), ctypes.c_int, i64p, ctypes.c_int, ctypes.c_int,
                                 f32p, ctypes.c_int]
    lib.stencil_apply.restype = ctypes.c_int
    lib.stencil_apply.argtypes = [vp, vp, vp, ctypes.c_int, vp]
    lib.stencil_plan_f64.restype = ctypes.c_int
    lib.stencil_plan_f64.argtypes = [ctypes.POINTER(vp), ctypes.c_int, i64p, ctypes.c_int, ctypes.c_int,
                                     ctypes.POINTER(ctypes.c_double), ctypes.c_int]
    lib.stencil_apply_f64.restype = ctypes.c_int
    lib.stencil_apply_f64.argtypes = [vp, vp, vp, ctypes.c_int, vp]
    lib.stencil_apply_host.restype = ctypes.c_int
    lib.stencil_apply_host.argtypes = [vp, vp, vp, ctypes.c_int, vp]
    lib.stencil_apply_planes.restype = ctypes.c_int
    lib.stencil_apply_planes.argtypes = [vp, vp, vp, ctypes.c_int64, ctypes.c_int64, vp]
    lib.stencil_apply_planes_f64.restype = ctypes.c_int
    lib.stencil_apply_planes_f64.argtypes = [vp, vp, vp, ctypes.c_int64, ctypes.c_int64, vp]
    lib.stencil_apply_static.restype = ctypes.c_int
    lib.stencil_apply_static.argtypes = [vp, vp, vp, ctypes.c_int, vp]
    lib.stencil_destroy.restype = ctypes.c_int
    lib.stencil_destroy.argtypes = [vp]
    lib.stencil_status_string.restype = ctypes.c_char_p
    lib.stencil_status_string.argtypes = [ctypes.c_int]
    lib.stencil_variant_name.restype = ctypes.c_char_p
    lib.stencil_variant_name.argtypes = [ctypes.c_int]
    lib.stencil_query_status.restype = ctypes.c_int
    lib.stencil_query_status.argtypes = [vp]
    lib.stencil_plan_set.restype = ctypes.c_int
    lib.stencil_plan_set.argtypes = [vp, ctypes.c_int, ctypes.c_int64]
    lib.stencil_plan_get.restype = ctypes.c_int
    lib.stencil_plan_get.argtypes = [vp, ctypes.c_int, i64p]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().stencil_status_string(int(status)).decode()


def variant_name(variant: int) -> str:
    return load().stencil_variant_name(int(variant)).decode()


# ---------------------------------------------------------------------------
# raw calls, same names and argument order as the C ABI; they return the status
# ---------------------------------------------------------------------------
def stencil_plan(dims: Sequence[int], radius: int, shape: int, weights: np.ndarray, boundary: int):
    """-> (status, handle).  ``weights``: dense float32 (2R+1)^ndim host array."""
    lib = load()
    w = np.ascontiguousarray(weights, dtype=np.float32)
    d = (ctypes.c_int64 * len(dims))(*[int(v) for v in dims])
    h = ctypes.c_void_p()
    rc = lib.stencil_plan(ctypes.byref(h), len(dims), d, int(radius), int(shape),
                          w.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), int(boundary))
    return rc, h


def stencil_plan_f64(dims: Sequence[int], radius: int, shape: int, weights: np.ndarray, boundary: int):
    """-> (status, handle) of an FP64 plan.  ``weights``: dense float64 (2R+1)^ndim host array."""
    lib = load()
    w = np.ascontiguousarray(weights, dtype=np.float64)
    d = (ctypes.c_int64 * len(dims))(*[int(v) for v in dims])
    h = ctypes.c_void_p()
    rc = lib.stencil_plan_f64(ctypes.byref(h), len(dims), d, int(radius), int(shape),
                              w.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), int(boundary))
    return rc, h


def stencil_apply_f64(plan, in_ptr: int, out_ptr: int, steps: int, stream: int = 0) -> int:
    """``in_ptr`` / ``out_ptr``: device addresses of float64 grids."""
    return load().stencil_apply_f64(plan, ctypes.c_void_p(in_ptr), ctypes.c_void_p(out_ptr), int(steps),
                                    ctypes.c_void_p(stream))


def stencil_apply(plan, in_ptr: int, out_ptr: int, steps: int, stream: int = 0) -> int:
    """``in_ptr`` / ``out_ptr``: device addresses; ``stream``: a cudaStream_t value."""
    return load().stencil_apply(plan, ctypes.c_void_p(in_ptr), ctypes.c_void_p(out_ptr), int(steps),
                                ctypes.c_void_p(stream))


def stencil_apply_host(plan, in_ptr: int, out_ptr: int, steps: int, stream: int = 0) -> int:
    """``in_ptr`` / ``out_ptr``: host addresses (pinned memory recommended)."""
    return load().stencil_apply_host(plan, ctypes.c_void_p(in_ptr), ctypes.c_void_p(out_ptr),
                                     int(steps), ctypes.c_void_p(stream))


def stencil_apply_planes(plan, in_ptr: int, out_ptr: int, z_begin: int, z_end: int, stream: int = 0) -> int:
    """One sweep restricted to the output planes [z_begin, z_end) of a 3D grid (rows of a 2D grid)."""
    return load().stencil_apply_planes(plan, ctypes.c_void_p(in_ptr), ctypes.c_void_p(out_ptr), int(z_begin),
                                       int(z_end), ctypes.c_void_p(stream))


def stencil_apply_planes_f64(plan, in_ptr: int, out_ptr: int, z_begin: int, z_end: int, stream: int = 0) -> int:
    """The same for an FP64 plan."""
    return load().stencil_apply_planes_f64(plan, ctypes.c_void_p(in_ptr), ctypes.c_void_p(out_ptr), int(z_begin),
                                           int(z_end), ctypes.c_void_p(stream))


def stencil_apply_static(plan, in_ptr: int, out_ptr: int, steps: int, stream: int = 0) -> int:
    """Like ``stencil_apply`` but never allocates device memory: the scratch is
    a fixed array inside the library, so grids above ``STATIC_MAX_POINTS`` are
    refused with ``ERR_TOO_LARGE``.  For callers that cannot call cudaMalloc
    where they run the sweep (all memory already in their own pool, or no room
    for the stall an allocation causes).  Calls share that one array: do not let
    two of them overlap on the GPU."""
    return load().stencil_apply_static(plan, ctypes.c_void_p(in_ptr), ctypes.c_void_p(out_ptr), int(steps),
                                       ctypes.c_void_p(stream))


def stencil_destroy(plan) -> int:
    return load().stencil_destroy(plan)


def stencil_query_status(plan) -> int:
    return load().stencil_query_status(plan)


def stencil_plan_set(plan, key: int, value: int) -> int:
    return load().stencil_plan_set(plan, int(key), int(value))


def stencil_plan_get(plan, key: int):
    v = ctypes.c_int64(0)
    rc = load().stencil_plan_get(plan, int(key), ctypes.byref(v))
    return rc, int(v.value)


# ---------------------------------------------------------------------------
# a small convenience wrapper that raises on errors
# ---------------------------------------------------------------------------
class Plan:
    """Owns one ``stencil_plan_t``.  ``apply`` takes device pointers (ints) or
    objects with ``data_ptr()`` such as torch CUDA tensors."""

    def __init__(self, dims, radius: int, shape: int, weights: np.ndarray, boundary: int = ZERO,
                 variant: Optional[int] = None, **knobs):
        self.f64 = np.asarray(weights).dtype == np.float64     # float64 weights make an FP64 plan
        rc, h = (stencil_plan_f64 if self.f64 else stencil_plan)(dims, radius, shape, weights, boundary)
        if rc != OK:
            raise StencilError(rc, "stencil_plan_f64" if self.f64 else "stencil_plan")
        self._h = h
        self.dims = tuple(int(d) for d in dims)
        self.npoints = int(np.prod(self.dims))
        if variant is not None:
            self.set(KEY_VARIANT, variant)
        keys = {"tile_y": KEY_TILE_Y, "chunk_z": KEY_CHUNK_Z, "stages": KEY_STAGES,
                "fuse_steps": KEY_FUSE_STEPS, "tile_x": KEY_TILE_X, "streaming_store": KEY_STREAMING_STORE,
                "rows_per_thread": KEY_ROWS_PER_THREAD, "chain_launches": KEY_CHAIN_LAUNCHES, "fused_tile_y": KEY_FUSED_TILE_Y,
                "periodic_route": KEY_PERIODIC_ROUTE}
        for name, value in knobs.items():
            if value is not None:
                self.set(keys[name], value)

    @classmethod
    def for_workload(cls, wk, **kw) -> "Plan":
        return cls(wk.dims, wk.radius, wk.shape, wk.weights(), wk.boundary, **kw)

    def set(self, key: int, value: int) -> None:
        rc = stencil_plan_set(self._h, key, value)
        if rc != OK:
            raise StencilError(rc, f"stencil_plan_set(key={key}, value={value})")

    def get(self, key: int) -> int:
        rc, v = stencil_plan_get(self._h, key)
        if rc != OK:
            raise StencilError(rc, f"stencil_plan_get(key={key})")
        return v

    @property
    def variant(self) -> str:
        return variant_name(self.get(KEY_VARIANT))

    @property
    def launches(self) -> int:
        return self.get(KEY_LAUNCHES)

    @staticmethod
    def _ptr(x) -> int:
        return int(x.data_ptr()) if hasattr(x, "data_ptr") else int(x)

    def apply(self, src, dst, steps: int = 1, stream: int = 0) -> None:
        fn = stencil_apply_f64 if self.f64 else stencil_apply
        rc = fn(self._h, self._ptr(src), self._ptr(dst), steps, stream)
        if rc != OK:
            raise StencilError(rc, "stencil_apply_f64" if self.f64 else "stencil_apply")

    def apply_planes(self, src, dst, z_begin: int, z_end: int, stream: int = 0) -> None:
        fn = stencil_apply_planes_f64 if self.f64 else stencil_apply_planes
        rc = fn(self._h, self._ptr(src), self._ptr(dst), z_begin, z_end, stream)
        if rc != OK:
            raise StencilError(rc, "stencil_apply_planes_f64" if self.f64 else "stencil_apply_planes")

    def apply_static(self, src, dst, steps: int = 1, stream: int = 0) -> None:
        rc = stencil_apply_static(self._h, self._ptr(src), self._ptr(dst), steps, stream)
        if rc != OK:
            raise StencilError(rc, "stencil_apply_static")

    def apply_host(self, src, dst, steps: int = 1, stream: int = 0) -> None:
        rc = stencil_apply_host(self._h, self._ptr(src), self._ptr(dst), steps, stream)
        if rc != OK:
            raise StencilError(rc, "stencil_apply_host")

    def query_status(self) -> int:
        return stencil_query_status(self._h)

    def destroy(self) -> None:
        if self._h is not None and self._h.value:
            rc = stencil_destroy(self._h)
            self._h = None
            if rc != OK:
                raise StencilError(rc, "stencil_destroy")

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.destroy()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
