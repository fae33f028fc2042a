"""ctypes front end of the plain-C oracle (``stencil_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The C file is the oracle: a loop nest that evaluates
``out[p] = sum_o w[o] * in[p+o]`` (the zero-padded, stride-1 cross-correlation
that the paper's case-study protocol equates with its box stencil), in double,
rounded to float32 once per step.  This wrapper compiles it with gcc on first
use and marshals numpy arrays; it adds no arithmetic.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

ZERO = 0
PERIODIC = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "stencil_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_stencil.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc -O2 -fopenmp) next to its source."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                   "-ffp-contract=off", "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64p = ctypes.POINTER(ctypes.c_int64)
        f32p = ctypes.POINTER(ctypes.c_float)
        lib.oracle_stencil_apply.restype = ctypes.c_int
        lib.oracle_stencil_apply.argtypes = [ctypes.c_int, i64p, ctypes.c_int, f32p,
                                             ctypes.c_int, ctypes.c_int, f32p, f32p]
        lib.oracle_stencil_points.restype = ctypes.c_int
        lib.oracle_stencil_points.argtypes = [ctypes.c_int, i64p, ctypes.c_int, f32p,
                                              ctypes.c_int, f32p, ctypes.c_int64, i64p, f32p]
        f64p = ctypes.POINTER(ctypes.c_double)
        lib.oracle_stencil_apply_f64.restype = ctypes.c_int
        lib.oracle_stencil_apply_f64.argtypes = [ctypes.c_int, i64p, ctypes.c_int, f64p,
                                                 ctypes.c_int, ctypes.c_int, f64p, f64p]
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _check(weights: np.ndarray, field: np.ndarray):
    if field.dtype != weights.dtype or field.dtype not in (np.float32, np.float64):
        raise TypeError("oracle takes float32 weights with float32 fields, or float64 with float64")
    ndim = field.ndim
    if ndim not in (2, 3) or weights.ndim != ndim:
        raise ValueError("field and weights must both be 2D or both 3D")
    side = weights.shape[0]
    if side % 2 != 1 or side < 3 or any(s != side for s in weights.shape):
        raise ValueError("weights must be a dense (2R+1)^ndim array with R >= 1")
    return ndim, (side - 1) // 2


def _f32p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _f64p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def apply(field: np.ndarray, weights: np.ndarray, boundary: int = ZERO, steps: int = 1) -> np.ndarray:
    """``steps``-fold sweep of ``field`` with dense ``weights``; returns a new array.
    float32 arrays use the double-accumulating oracle, float64 arrays the long-double one."""
    field = np.ascontiguousarray(field)
    weights = np.ascontiguousarray(weights)
    ndim, R = _check(weights, field)
    dims = (ctypes.c_int64 * ndim)(*field.shape)
    out = np.empty_like(field)
    if field.dtype == np.float64:
        rc = _load().oracle_stencil_apply_f64(ndim, dims, R, _f64p(weights), int(boundary), int(steps),
                                              _f64p(field), _f64p(out))
        if rc != 0:
            raise RuntimeError(f"oracle_stencil_apply_f64 failed ({rc})")
        return out
    rc = _load().oracle_stencil_apply(ndim, dims, R, _f32p(weights), int(boundary), int(steps),
                                      _f32p(field), _f32p(out))
    if rc != 0:
        raise RuntimeError(f"oracle_stencil_apply failed ({rc})")
    return out


def apply_points(field: np.ndarray, weights: np.ndarray, flat_index: np.ndarray,
                 boundary: int = ZERO) -> np.ndarray:
    """One sweep evaluated only at ``flat_index`` (C-order flat indices)."""
    field = np.ascontiguousarray(field)
    weights = np.ascontiguousarray(weights)
    ndim, R = _check(weights, field)
    if field.dtype != np.float32:
        raise TypeError("apply_points is float32 only")
    idx = np.ascontiguousarray(flat_index, dtype=np.int64)
    dims = (ctypes.c_int64 * ndim)(*field.shape)
    out = np.empty(idx.shape, dtype=np.float32)
    rc = _load().oracle_stencil_points(ndim, dims, R, _f32p(weights), int(boundary), _f32p(field),
                                       idx.size, idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                                       _f32p(out))
    if rc != 0:
        raise RuntimeError(f"oracle_stencil_points failed ({rc})")
    return out
