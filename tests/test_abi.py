"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every symbol the header declares, validates arguments, and refuses to compute
without a device instead of falling back to anything."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2608_21157_b200 import binding as b
from paper_2608_21157_b200 import build as build_mod
from paper_2608_21157_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()
    b.load()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "stencil.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"STENCIL_API\s+[\w\s\*]+?\b(stencil_\w+)\s*\(", text)))


def test_header_and_binding_list_the_same_symbols():
    assert _declared_symbols() == sorted(b.EXPORTS)


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(b.LIB_PATH)
    for name in _declared_symbols():
        assert getattr(lib, name) is not None


def test_binding_does_not_import_the_oracle():
    import paper_2608_21157_b200
    pkg_dir = os.path.dirname(paper_2608_21157_b200.__file__)
    for dirpath, _, files in os.walk(pkg_dir):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src
                assert "stencil_oracle" not in src
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2608_21157_b200" not in src and "stencil.h" not in src


def test_status_and_variant_strings():
    assert b.status_string(b.OK) == "ok"
    for code in (b.ERR_INVALID, b.ERR_UNSUPPORTED, b.ERR_CUDA, b.ERR_ALLOC, b.ERR_TIMEOUT, 12345):
        assert isinstance(b.status_string(code), str) and b.status_string(code)
    assert b.variant_name(b.VARIANT_GENERIC) == "generic"
    assert b.variant_name(b.VARIANT_STREAM) == "stream"


def _w(ndim, R):
    return wl.random_box_weights(ndim, R, 1)


@pytest.mark.parametrize("dims,R,shape,boundary,want", [
    ((8, 8), 0, b.BOX, b.ZERO, b.ERR_INVALID),
    ((8, 8), 9, b.BOX, b.ZERO, b.ERR_UNSUPPORTED),
    ((8, 0), 1, b.BOX, b.ZERO, b.ERR_INVALID),
    ((8, -3, 4), 1, b.BOX, b.ZERO, b.ERR_INVALID),
    ((8, 8), 1, 7, b.ZERO, b.ERR_INVALID),
    ((8, 8), 1, b.BOX, 5, b.ERR_INVALID),
    ((8,), 1, b.BOX, b.ZERO, b.ERR_INVALID),
    ((4, 4, 4, 4), 1, b.BOX, b.ZERO, b.ERR_INVALID),
])
def test_plan_rejects_bad_arguments(dims, R, shape, boundary, want):
    ndim = min(max(len(dims), 2), 3)
    rc, h = b.stencil_plan(dims, R, shape, _w(ndim, max(R, 1)), boundary)
    assert rc == want
    assert not h.value


def test_plan_null_pointers():
    lib = b.load()
    h = ctypes.c_void_p()
    d = (ctypes.c_int64 * 2)(4, 4)
    w = _w(2, 1)
    wp = w.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    assert lib.stencil_plan(None, 2, d, 1, b.BOX, wp, b.ZERO) == b.ERR_INVALID
    assert lib.stencil_plan(ctypes.byref(h), 2, None, 1, b.BOX, wp, b.ZERO) == b.ERR_INVALID
    assert lib.stencil_plan(ctypes.byref(h), 2, d, 1, b.BOX, None, b.ZERO) == b.ERR_INVALID


def test_star_promise_is_checked():
    w = _w(3, 1)                                   # dense box weights are not a star
    rc, h = b.stencil_plan((8, 8, 8), 1, b.STAR, w, b.ZERO)
    assert rc == b.ERR_INVALID and not h.value
    rc, h = b.stencil_plan((8, 8, 8), 1, b.STAR, wl.star_weights(3, 1, -6.0, [1.0]), b.ZERO)
    assert rc == b.OK
    assert b.stencil_destroy(h) == b.OK


def test_variant_selection_rules():
    star = wl.star_weights(3, 1, -6.0, [1.0])
    with b.Plan((64, 64, 64), 1, b.STAR, star, b.ZERO) as p:
        assert p.variant == "stream"
        p.set(b.KEY_VARIANT, b.VARIANT_GENERIC)
        assert p.variant == "generic"
    with b.Plan((64, 64, 66), 1, b.STAR, star, b.ZERO) as p:       # nx % 4 != 0: swept between grids with padded rows
        assert p.variant == "stream"
        assert p.get(b.KEY_FUSE_STEPS) == 1         # no temporal blocking over padded rows
    with b.Plan((64, 64, 64), 6, b.STAR, wl.star_weights(3, 6, -6.0, [1.0] * 6), b.ZERO) as p:
        assert p.variant == "stream"                # the wide stars run on the tiled 3D kernel (8-column halos)
    with b.Plan((64, 64), 6, b.STAR, wl.star_weights(2, 6, -6.0, [1.0] * 6), b.ZERO) as p:
        assert p.variant == "stream" and p.get(b.KEY_FUSE_STEPS) == 1     # also in 2D; no fused kernel for them
    with b.Plan((64, 64), 5, b.BOX, wl.random_box_weights(2, 5, 4), b.ZERO) as p:
        assert p.variant == "generic"               # boxes beyond radius 4 are not tiled
    with b.Plan((8, 64, 64), 6, b.STAR, wl.star_weights(3, 6, -6.0, [1.0] * 6), b.PERIODIC) as p:
        assert p.variant == "generic"               # periodic wide star on a grid thinner than 2R
    with b.Plan((64, 64, 66), 3, b.BOX, wl.random_box_weights(3, 3, 4), b.ZERO) as p:
        assert p.variant == "generic"               # radius beyond the tiled kernels
        with pytest.raises(b.StencilError) as e:
            p.set(b.KEY_VARIANT, b.VARIANT_STREAM)
        assert e.value.status == b.ERR_UNSUPPORTED
        assert p.variant == "generic"
    with b.Plan((64, 64, 64), 1, b.STAR, star, b.PERIODIC) as p:
        assert p.variant == "stream"                # swept from a padded copy with wrapped halos
        assert p.get(b.KEY_FUSE_STEPS) == 1         # rows of 64 points are too narrow for the fused regions
    with b.Plan((64, 64, 256), 1, b.STAR, star, b.PERIODIC) as p:
        assert p.variant == "stream" and p.get(b.KEY_FUSE_STEPS) == 2     # periodic grids fuse like zero-boundary ones
    with b.Plan((3, 64, 256), 1, b.STAR, star, b.PERIODIC) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1         # ... when every extent holds both shells of depth T * R
    with b.Plan((64, 64, 62), 1, b.STAR, star, b.PERIODIC) as p:
        assert p.variant == "generic"
        with pytest.raises(b.StencilError) as e:
            p.set(b.KEY_VARIANT, b.VARIANT_STREAM)
        assert e.value.status == b.ERR_UNSUPPORTED
    with b.Plan((64, 64), 1, b.STAR, wl.star_weights(2, 1, -4.0, [1.0]), b.ZERO) as p:
        assert p.variant in ("generic", "stream")
    with b.Plan((64, 64, 64), 1, b.STAR, star, b.ZERO) as p:
        with pytest.raises(b.StencilError):
            p.set(b.KEY_TILE_Y, 7)
        with pytest.raises(b.StencilError):
            p.set(b.KEY_STAGES, 99)
        with pytest.raises(b.StencilError):
            p.set(12345, 1)


def test_apply_argument_checks_and_no_cpu_fallback():
    with b.Plan((8, 8, 8), 1, b.BOX, _w(3, 1), b.ZERO) as p:
        n = 8 * 8 * 8 * 4
        base = 1 << 30
        assert b.stencil_apply(p._h, 0, base, 1) == b.ERR_INVALID            # NULL in
        assert b.stencil_apply(p._h, base, 0, 1) == b.ERR_INVALID            # NULL out
        assert b.stencil_apply(p._h, base, base, 1) == b.ERR_INVALID         # in == out
        assert b.stencil_apply(p._h, base, base + n - 16, 1) == b.ERR_INVALID  # overlap
        assert b.stencil_apply(p._h, base + 4, base + 2 * n, 1) == b.ERR_INVALID  # misaligned
        assert b.stencil_apply(p._h, base, base + 2 * n, -1) == b.ERR_INVALID
        assert b.stencil_apply(None, base, base + 2 * n, 1) == b.ERR_INVALID
        import torch
        if not torch.cuda.is_available():
            # valid arguments but no device: the library must refuse, not compute on the CPU
            assert b.stencil_apply(p._h, base, base + 2 * n, 1) == b.ERR_CUDA
            a = np.zeros((8, 8, 8), np.float32)
            o = np.zeros_like(a)
            assert b.stencil_apply_host(p._h, a.ctypes.data, o.ctypes.data, 1) == b.ERR_CUDA


def test_destroy_null_is_ok_and_get_counters():
    assert b.stencil_destroy(None) == b.OK
    with b.Plan((8, 8, 8), 1, b.BOX, _w(3, 1), b.ZERO) as p:
        assert p.launches == 0
        assert p.get(b.KEY_SCRATCH_BYTES) == 0
        assert p.query_status() == b.OK


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        b.load()


def test_fuse_knob_rules():
    """Which iterated applies fuse time steps by default, and with which region (host logic only)."""
    star = wl.star_weights(3, 1, 0.4, [0.1])
    with b.Plan((64, 64, 1000), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2 and p.get(b.KEY_TILE_X) == 384      # three 384-wide regions: 87 % of their lanes
    with b.Plan((64, 64, 1024), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2 and p.get(b.KEY_TILE_X) == 384      # three regions store 376 columns each: 89 %
        assert p.get(b.KEY_FUSED_TILE_Y) == 20
        p.set(b.KEY_FUSE_STEPS, 4)
        assert p.get(b.KEY_FUSE_STEPS) == 4
    with b.Plan((64, 64, 768), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1         # three 384-wide regions 67 %, two 512-wide ones 75 %
    with b.Plan((64, 64, 320), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2 and p.get(b.KEY_TILE_X) == 384      # 83 % of a 384-wide region
    with b.Plan((64, 64, 260), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2 and p.get(b.KEY_TILE_X) == 384      # pays off from 257 points on
    with b.Plan((64, 64, 400), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1         # 78 % of a 512-wide region
    with b.Plan((64, 64, 896), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2 and p.get(b.KEY_TILE_X) == 384      # three regions, 78 %
    with b.Plan((64, 64, 512), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2 and p.get(b.KEY_FUSED_TILE_Y) == 16   # one 512-wide region per row
    with b.Plan((64, 64, 448), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2
    with b.Plan((64, 64, 64), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1         # half of a 128-wide region's lanes would idle
    with b.Plan((64, 64, 200), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1         # 78 % of a 256-wide region
    with b.Plan((64, 64, 128), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2 and p.get(b.KEY_TILE_X) == 128     # too few CTAs for three levels
    with b.Plan((512, 512, 128), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 3 and p.get(b.KEY_TILE_X) == 128     # narrow regions: three levels fit
        p.set(b.KEY_FUSE_STEPS, 2)
        assert p.get(b.KEY_FUSE_STEPS) == 2 and p.get(b.KEY_TILE_X) == 128
    with b.Plan((64, 64, 256), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) >= 2         # iterated applies fuse by default
        assert p.get(b.KEY_TILE_X) == 256 and p.get(b.KEY_FUSED_TILE_Y) == 16
        p.set(b.KEY_FUSE_STEPS, 1)
        assert p.get(b.KEY_FUSE_STEPS) == 1
        with pytest.raises(b.StencilError):
            p.set(b.KEY_FUSE_STEPS, 7)
    with b.Plan((64, 448, 256), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2         # from 448 rows on the 256-wide regions are 32 rows high
        assert p.get(b.KEY_TILE_X) == 256 and p.get(b.KEY_FUSED_TILE_Y) == 32
        p.set(b.KEY_FUSED_TILE_Y, 16)
        assert p.get(b.KEY_FUSED_TILE_Y) == 16
    with b.Plan((64, 444, 256), 1, b.STAR, star, b.ZERO) as p:
        assert p.get(b.KEY_FUSED_TILE_Y) == 16
    with b.Plan((64, 64, 64), 1, b.BOX, wl.random_box_weights(3, 1, 3), b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1         # no fused kernel for box stencils
        with pytest.raises(b.StencilError):
            p.set(b.KEY_VARIANT, b.VARIANT_FUSED)


def test_fp64_variant_selection_rules():
    """Which FP64 requests the tiled kernels take (host logic only)."""
    def plan(dims, R, box, boundary):
        nd = len(dims)
        w = (wl.random_box_weights if box else wl.random_star_weights)(nd, R, 3, np.float64)
        return b.Plan(dims, R, b.BOX if box else b.STAR, w, boundary)
    tiled = [((64, 64), 4, True, b.ZERO), ((64, 64), 4, False, b.PERIODIC), ((33, 65), 3, True, b.ZERO),
             ((32, 32, 32), 2, True, b.ZERO), ((32, 32, 32), 4, False, b.PERIODIC), ((8, 9, 31), 1, True, b.ZERO),
             ((32, 32, 32), 5, False, b.ZERO), ((64, 64), 8, False, b.PERIODIC), ((16, 16, 16), 8, False, b.PERIODIC)]
    generic = [((64, 64), 5, True, b.ZERO), ((32, 32, 32), 3, True, b.ZERO), ((32, 32, 12), 7, False, b.PERIODIC),
               ((32, 32, 31), 1, False, b.PERIODIC), ((64, 63), 1, False, b.PERIODIC)]
    for args in tiled:
        with plan(*args) as p:
            assert p.f64 and p.variant == "stream", args
    for args in generic:
        with plan(*args) as p:
            assert p.f64 and p.variant == "generic", args
            with pytest.raises(b.StencilError) as e:
                p.set(b.KEY_VARIANT, b.VARIANT_STREAM)
            assert e.value.status == b.ERR_UNSUPPORTED


def test_fuse_rules_2d():
    """Iterated 2D applies fuse T steps per pass for the operators with a fused kernel (host logic only)."""
    for R, box, T in [(1, False, 4), (1, True, 4), (2, False, 3), (2, True, 2), (3, False, 2), (4, False, 2)]:
        w = wl.random_box_weights(2, R, 3) if box else wl.random_star_weights(2, R, 3)
        with b.Plan((64, 128), R, b.BOX if box else b.STAR, w, b.ZERO) as p:
            assert p.get(b.KEY_FUSE_STEPS) == T
            p.set(b.KEY_FUSE_STEPS, 1)
            assert p.get(b.KEY_FUSE_STEPS) == 1
            p.set(b.KEY_FUSE_STEPS, T)
            assert p.get(b.KEY_FUSE_STEPS) == T
            with pytest.raises(b.StencilError) as e:
                p.set(b.KEY_FUSE_STEPS, T + 1)
            assert e.value.status == b.ERR_UNSUPPORTED and p.get(b.KEY_FUSE_STEPS) == T
            p.set(b.KEY_FUSE_STEPS, 0)
            assert p.get(b.KEY_FUSE_STEPS) == T
        with b.Plan((64, 128), R, b.BOX if box else b.STAR, w, b.PERIODIC) as p:
            assert p.get(b.KEY_FUSE_STEPS) == T         # a periodic grid fuses too (its shell is rewritten after a pass) ...
        with b.Plan((2 * T * R - 1, 128), R, b.BOX if box else b.STAR, w, b.PERIODIC) as p:
            assert p.get(b.KEY_FUSE_STEPS) == 1         # ... when it holds both shells of depth T * R
        with b.Plan((64, 126), R, b.BOX if box else b.STAR, w, b.ZERO) as p:
            assert p.get(b.KEY_FUSE_STEPS) == 1         # rows that are not 16-byte multiples
    with b.Plan((64, 128), 3, b.BOX, wl.random_box_weights(2, 3, 3), b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1             # the 49-point box is bound by the FMA pipe: not fused
        with pytest.raises(b.StencilError):
            p.set(b.KEY_VARIANT, b.VARIANT_FUSED)


def test_fuse_rules_2d_fp64():
    for R, box, T in [(1, False, 4), (1, True, 4), (2, False, 3), (2, True, 2)]:
        w = (wl.random_box_weights if box else wl.random_star_weights)(2, R, 3, np.float64)
        with b.Plan((64, 128), R, b.BOX if box else b.STAR, w, b.ZERO) as p:
            assert p.f64 and p.get(b.KEY_FUSE_STEPS) == T
            p.set(b.KEY_FUSE_STEPS, 1)
            assert p.get(b.KEY_FUSE_STEPS) == 1
            with pytest.raises(b.StencilError):
                p.set(b.KEY_FUSE_STEPS, T + 1)
            p.set(b.KEY_FUSE_STEPS, 0)
            assert p.get(b.KEY_FUSE_STEPS) == T
        with b.Plan((64, 127), R, b.BOX if box else b.STAR, w, b.ZERO) as p:
            assert p.get(b.KEY_FUSE_STEPS) == 1         # odd rows run between padded-row grids, unfused
    w = wl.random_star_weights(2, 3, 3, np.float64)
    with b.Plan((64, 128), 3, b.STAR, w, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1             # radius 3 needs two neighbour lanes: no FP64 cascade
    w = wl.random_star_weights(3, 1, 3, np.float64)
    with b.Plan((32, 32, 64), 1, b.STAR, w, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1             # FP64 3D: a 64-wide row fills half a 128-wide region
        p.set(b.KEY_FUSE_STEPS, 2)                      # ... but the caller may ask for fused passes
        assert p.get(b.KEY_FUSE_STEPS) == 2
        with pytest.raises(b.StencilError):
            p.set(b.KEY_FUSE_STEPS, 4)                  # FP64 3D passes fuse two or three steps
        p.set(b.KEY_FUSE_STEPS, 0)
        assert p.get(b.KEY_FUSE_STEPS) == 1
    with b.Plan((32, 32, 256), 1, b.STAR, w, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 2             # one 256-wide region spans the row
    w2 = wl.random_star_weights(3, 2, 3, np.float64)
    with b.Plan((32, 32, 256), 2, b.STAR, w2, b.ZERO) as p:
        assert p.get(b.KEY_FUSE_STEPS) == 1             # radius 1 only
        with pytest.raises(b.StencilError):
            p.set(b.KEY_FUSE_STEPS, 2)


def test_device_key_reads_minus_one_before_the_first_apply():
    w = wl.star_weights(2, 1, -4.0, [1.0])
    rc, h = b.stencil_plan((16, 16), 1, b.STAR, w, b.ZERO)
    assert rc == b.OK
    rc, dev = b.stencil_plan_get(h, b.KEY_DEVICE)
    assert rc == b.OK and dev == -1
    assert b.stencil_destroy(h) == b.OK


@pytest.mark.gpu
def test_a_plan_stays_on_the_device_of_its_first_apply():
    """The plan's status word, taps, scratch grids and tensor maps live on the device that was
    current at the first apply; an apply with another device current is refused."""
    import torch
    w = wl.star_weights(2, 1, -4.0, [1.0])
    with b.Plan((64, 128), 1, b.STAR, w, b.ZERO) as p:
        with torch.cuda.device(0):
            src = torch.zeros((64, 128), dtype=torch.float32, device="cuda:0")
            dst = torch.empty_like(src)
            p.apply(src, dst, 1, 0)
            assert p.get(b.KEY_DEVICE) == 0
        if torch.cuda.device_count() < 2:
            pytest.skip("needs two visible GPUs to make another device current")
        with torch.cuda.device(1):
            assert b.stencil_apply(p._h, src.data_ptr(), dst.data_ptr(), 1, 0) == b.ERR_INVALID
        with torch.cuda.device(0):
            p.apply(src, dst, 1, 0)
            assert p.query_status() == b.OK


def test_header_is_plain_c_and_links_against_the_library(tmp_path):
    """include/stencil.h compiles as C99 with a strict compiler, and a C program that uses only the header
    links against the library and gets the documented statuses back (host-side checks only: no GPU needed)."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "use_abi.c"
    src.write_text(r'''
#include "stencil.h"
#include <stdio.h>
int main(void) {
    stencil_plan_t p = (stencil_plan_t)0x1;
    int64_t dims[3] = {8, 8, 8};
    float w[27];
    for (int i = 0; i < 27; ++i) w[i] = 0.0f;
    w[13] = -6.0f; w[4] = w[10] = w[12] = w[14] = w[16] = w[22] = 1.0f;
    if (stencil_plan(&p, 3, dims, 0, STENCIL_STAR, w, STENCIL_ZERO) != STENCIL_ERR_INVALID || p != 0) return 1;
    if (stencil_plan(&p, 3, dims, 9, STENCIL_STAR, w, STENCIL_ZERO) != STENCIL_ERR_UNSUPPORTED) return 2;
    w[0] = 1.0f;                                   /* an off-axis weight breaks the STAR promise */
    if (stencil_plan(&p, 3, dims, 1, STENCIL_STAR, w, STENCIL_ZERO) != STENCIL_ERR_INVALID) return 3;
    if (stencil_plan(&p, 3, dims, 1, STENCIL_BOX, w, STENCIL_ZERO) != STENCIL_OK || p == 0) return 4;
    int64_t v = -1;
    if (stencil_plan_get(p, STENCIL_KEY_LAUNCHES, &v) != STENCIL_OK || v != 0) return 5;
    if (stencil_plan_get(p, STENCIL_KEY_DEVICE, &v) != STENCIL_OK || v != -1) return 6;
    if (stencil_apply(p, 0, 0, 1, 0) != STENCIL_ERR_INVALID) return 7;
    if (stencil_query_status(p) != STENCIL_OK) return 8;
    if (stencil_destroy(p) != STENCIL_OK || stencil_destroy(0) != STENCIL_OK) return 9;
    puts(stencil_status_string(STENCIL_ERR_TIMEOUT));
    return 0;
}
''')
    exe = tmp_path / "use_abi"
    lib_dir = os.path.dirname(b.LIB_PATH)
    cmd = [gcc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(root, "include"),
           str(src), "-o", str(exe), "-L", lib_dir, "-l:libstencil_b200.so", f"-Wl,-rpath,{lib_dir}"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 0, f"step {r.returncode} of the C program failed"
    assert "wait" in r.stdout
