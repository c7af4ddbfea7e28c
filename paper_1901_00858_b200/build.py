"""Builds libhgc.so (the C-ABI CUDA library) and libhgc_debug.so (the same sources with -DHGC_DEBUG:
every hand-addressed global access tested against the call's tensors) in-tree with nvcc for sm_100a.

    python -m paper_1901_00858_b200.build [--force] [--verbose] [--no-debug]
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libhgc.so")
DEBUG_LIB = os.path.join(HERE, "libhgc_debug.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", "-O3", "-lineinfo",
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + [os.path.join(ROOT, "include", "hgc.h"), __file__]
    return any(os.path.getmtime(p) > t for p in deps)


def _compile(lib: str, extra: list, verbose: bool) -> None:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + [
        "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", tmp] + sources()
    subprocess.check_call(cmd)
    os.replace(tmp, lib)


def build(force: bool = False, verbose: bool = False, debug: bool = True) -> str:
    if force or _stale(LIB):
        _compile(LIB, [], verbose)
    if debug and (force or _stale(DEBUG_LIB)):
        _compile(DEBUG_LIB, ["-DHGC_DEBUG"], verbose)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--no-debug" not in sys.argv))
