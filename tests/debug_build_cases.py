"""Run by tests/test_debug_build_gpu.py in a process of its own with STENCIL_B200_DEBUG=1, so that the binding
loads the debug build of the library: default plans of every tiled kernel family against the oracle with the store
checks on (none may fire), then the same plans with the checks told that the grid is shorter than it is (they
must fire, skip the stores and leave everything before them right).  Exits non-zero on the first failure."""
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import oracle                                                   # noqa: E402
from paper_2608_21157_b200 import binding as b                  # noqa: E402
from paper_2608_21157_b200 import workloads as wl               # noqa: E402

# (dims, radius, box, boundary, dtype, steps): one case per tiled kernel family and route
CASES = [
    ((40, 70, 256), 1, False, b.ZERO, np.float32, 1),           # 3D stream, star
    ((24, 50, 132), 1, True, b.ZERO, np.float32, 1),            # 3D stream, box
    ((30, 40, 260), 4, False, b.ZERO, np.float32, 1),           # 3D stream, radius 4
    ((20, 37, 256), 1, False, b.PERIODIC, np.float32, 1),       # 3D stream that wraps inside the kernel
    ((40, 50, 256), 1, False, b.ZERO, np.float32, 5),           # 3D fused passes (256 x 16 regions) + one sweep
    ((24, 460, 256), 1, False, b.ZERO, np.float32, 4),          # 256 x 32 regions
    ((36, 70, 512), 1, False, b.PERIODIC, np.float32, 4),       # 512-wide regions, periodic passes
    ((300, 520), 1, False, b.ZERO, np.float32, 1),              # 2D rows, star
    ((200, 1028), 3, True, b.ZERO, np.float32, 2),              # 2D rows, the paper's 49-point box
    ((260, 1024), 1, False, b.ZERO, np.float32, 9),             # 2D fused cascade
    ((24, 40, 256), 1, False, b.ZERO, np.float64, 1),           # FP64 3D stream
    ((24, 48, 256), 1, False, b.ZERO, np.float64, 4),           # FP64 3D fused passes
    ((200, 512), 3, True, b.ZERO, np.float64, 1),               # FP64 2D rows
    ((200, 512), 1, False, b.ZERO, np.float64, 8),              # FP64 2D fused cascade
]


def run(case, shrink):
    dims, R, box, boundary, dt, steps = case
    ndim = len(dims)
    w = (wl.random_box_weights if box else wl.random_star_weights)(ndim, R, 77, dt)
    a = wl.normal_field(dims, 78, dt)
    n = a.size
    src = torch.from_numpy(a).cuda()
    dst = torch.full_like(src, float("nan"))
    with b.Plan(dims, R, b.BOX if box else b.STAR, w, boundary) as p:
        assert p.variant == "stream", (case, p.variant)
        p.set(b.KEY_DEBUG_SHRINK, shrink)
        assert p.get(b.KEY_DEBUG_SHRINK) == shrink
        # (every launch of an iterated apply is checked against its own output buffer)
        p.apply(src, dst, steps, torch.cuda.current_stream().cuda_stream)
        status = p.query_status()
    got = dst.cpu().numpy().reshape(-1)
    want = oracle.apply(a, w, boundary, steps).reshape(-1)
    tol = wl.tolerance(w, float(np.abs(a).max()), steps)
    return status, got, want, tol, n


def main():
    assert b.DEBUG_BUILD and b.LIB_PATH.endswith("libstencil_b200_debug.so")
    for case in CASES:
        status, got, want, tol, n = run(case, 0)
        assert status == b.OK, f"{case}: a store check fired on a correct launch ({status})"
        err = float(np.max(np.abs(got - want)))
        assert err <= tol, f"{case}: {err:.3e} > {tol:.3e}"
    for case in CASES:
        steps = case[5]
        nx = case[0][-1]
        shrink = 2 * nx + 5
        status, got, want, tol, n = run(case, shrink)
        assert status == b.ERR_BOUNDS, f"{case}: stores past the claimed end went unnoticed ({status})"
        # a vector store that reaches past the claimed end is skipped as a whole (4 floats, 2 doubles)
        head = n - shrink - 4
        if steps == 1:
            assert np.isnan(got[n - shrink:]).all(), f"{case}: a store past the claimed end was not skipped"
            err = float(np.max(np.abs(got[:head] - want[:head])))
            assert err <= tol, f"{case}: points before the claimed end are wrong ({err:.3e})"
    print("debug build: all cases passed")


if __name__ == "__main__":
    main()
