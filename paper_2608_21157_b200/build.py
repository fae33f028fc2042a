"""Builds the CUDA library in-tree with nvcc for sm_100a.

    python -m paper_2608_21157_b200.build [--force] [--verbose]

The result, ``paper_2608_21157_b200/libstencil_b200.so``, is what the Python
binding loads.  nvcc cross-compiles, so no GPU is needed to build.  The host
side is split by kernel family (``csrc/host_*.cu`` and ``csrc/abi.cu``); the
units compile in parallel into ``paper_2608_21157_b200/build/`` and only those
whose sources changed are recompiled.

``--debug`` builds ``libstencil_b200_debug.so`` instead (objects in ``build_debug/``): the same sources with
``-DSTENCIL_DEBUG``, in which every global store of the tiled kernels is checked against the extent of the output
grid (a store outside it is skipped and reported by ``stencil_query_status``).  The binding loads it when the
environment variable ``STENCIL_B200_DEBUG`` is ``1``.
"""
from __future__ import annotations

import os
import re
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libstencil_b200.so")
OBJ_DEBUG = os.path.join(HERE, "build_debug")
LIB_DEBUG = os.path.join(HERE, "libstencil_b200_debug.so")
HEADER = os.path.join(os.path.dirname(HERE), "include", "stencil.h")
SOURCES = ["abi.cu", "host_common.cu", "host_stream.cu", "host_fused.cu", "host_rows2d.cu", "host_f64.cu",
           "host_periodic.cu"]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
         "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--expt-relaxed-constexpr"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; the CUDA library cannot be built")


def _includes(path: str, seen: set) -> set:
    """Files under csrc/ that `path` includes, directly or not."""
    if path in seen:
        return seen
    seen.add(path)
    with open(path) as f:
        for name in re.findall(r'^#include "([^"]+)"', f.read(), flags=re.M):
            dep = os.path.normpath(os.path.join(os.path.dirname(path), name))
            if os.path.exists(dep):
                _includes(dep, seen)
    return seen


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    obj_dir, lib = (OBJ_DEBUG, LIB_DEBUG) if debug else (OBJ, LIB)
    flags = FLAGS + (["-DSTENCIL_DEBUG"] if debug else [])
    os.makedirs(obj_dir, exist_ok=True)
    nvcc = _nvcc()
    jobs = []
    for s in SOURCES:
        src = os.path.join(CSRC, s)
        obj = os.path.join(obj_dir, s[:-3] + ".o")
        if force or _stale(obj, _includes(src, set()) | {HEADER}):
            jobs.append((src, obj))

    def compile_one(job):
        src, obj = job
        tmp = obj + f".tmp{os.getpid()}"
        cmd = [nvcc] + flags + (["-Xptxas", "-v"] if verbose else []) + ["-c", "-o", tmp, src]
        subprocess.run(cmd, check=True)
        os.replace(tmp, obj)

    if jobs:
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as pool:
            list(pool.map(compile_one, jobs))
    objs = [os.path.join(obj_dir, s[:-3] + ".o") for s in SOURCES]
    if force or jobs or _stale(lib, objs):
        tmp = lib + f".tmp{os.getpid()}"
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static",
                        "-o", tmp] + objs, check=True)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
