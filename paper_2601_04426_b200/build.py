"""Build libxg.so in tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libxg.so")
LIB_DEBUG = os.path.join(HERE, "libxg_dbg.so")      # the same sources with -DXG_DEBUG_BOUNDS
SOURCES = ["api.cu", "frontend.cpp", "pool.cpp"]
HEADERS = ["device_types.h", "frontend.h", "kernels.cuh", "pool.h", os.path.join("..", "..", "include", "xg.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    return "nvcc"


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    lib = LIB_DEBUG if debug_bounds else LIB
    if not force and not needs_build(lib):
        return lib
    tmp = lib + ".tmp%d" % os.getpid()
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--extended-lambda", "-shared", "-Xcompiler", "-fPIC", "-x", "cu",
           "-I", os.path.join(HERE, "..", "include"), "-I", CSRC]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if debug_bounds:
        cmd += ["-DXG_DEBUG_BOUNDS"]
    cmd += [os.path.join(CSRC, f) for f in SOURCES] + ["-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
