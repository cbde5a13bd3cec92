"""Builds ``libchicle.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_1909_04885_b200.build [--force] [--verbose] [--debug-bounds]

``--debug-bounds`` builds ``libchicle_bounds.so`` beside it with ``-DCHICLE_DEBUG_BOUNDS``: every index that the
solvers and the gap kernels load (visiting-order entries, row extents, entry ids, record directory entries, record sizes)
is checked before use; a failed check sets a status bit that the call returns as ``CHICLE_ERR_INTERNAL`` and the access
is skipped. Select it with ``CHICLE_LIB_PATH``.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libchicle.so")
LIB_BOUNDS = os.path.join(HERE, "libchicle_bounds.so")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    lib = LIB_BOUNDS if debug_bounds else LIB
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if debug_bounds:
        cmd += ["-DCHICLE_DEBUG_BOUNDS"]
    cmd += os.environ.get("CHICLE_NVCC_FLAGS", "").split()  # e.g. -DCHICLE_LA_TIMING: cycle counters around the look-ahead solver's phases, printed after every launch
    cmd += ["-o", tmp] + sources()
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
