"""The debug build of the library (``-DSTENCIL_DEBUG``): every global store of the tiled kernels is checked
against the extent of the output grid."""
import ctypes
import os
import subprocess
import sys

import numpy as np
import pytest

from paper_2608_21157_b200 import binding as b
from paper_2608_21157_b200 import build as build_mod
from paper_2608_21157_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_debug_library_builds_and_exports_the_same_symbols():
    lib = ctypes.CDLL(build_mod.build(debug=True))
    for name in b.EXPORTS:
        assert hasattr(lib, name), name


def test_the_release_build_has_no_store_checks_to_configure():
    w = wl.random_star_weights(3, 1, 5)
    with b.Plan((8, 8, 128), 1, b.STAR, w, b.ZERO) as p:
        with pytest.raises(b.StencilError) as e:
            p.set(b.KEY_DEBUG_SHRINK, 1)
        assert e.value.status == b.ERR_UNSUPPORTED
        with pytest.raises(b.StencilError):
            p.get(b.KEY_DEBUG_SHRINK)
    assert "debug" in b.status_string(b.ERR_BOUNDS)


@pytest.mark.gpu
def test_debug_build_checks_every_tiled_family():
    """Parity of every tiled kernel family with the checks on, and the checks firing (stores skipped, status
    STENCIL_ERR_BOUNDS, nothing faults) when told that the grid ends early: see tests/debug_build_cases.py."""
    build_mod.build(debug=True)
    env = dict(os.environ, STENCIL_B200_DEBUG="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "debug_build_cases.py")], env=env,
                       capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "all cases passed" in r.stdout
