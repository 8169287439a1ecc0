"""Builds the CUDA library in-tree with nvcc for sm_100a.

    python -m paper_2411_18462_b200.build [--force] [--verbose] [--debug]

--debug builds csrc/libsvip_debug.so instead: the same library with bounds checks on every load of
logits (out-of-range loads are skipped and reported in the status word) and NVTX ranges around the
entry points.  Point SVIP_LIBRARY at it to run anything against the checked build.

The shared object is written next to the sources (csrc/libsvip.so) so that it
travels with the source tree; it is never installed into site-packages.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
INCLUDE = os.path.join(os.path.dirname(PKG), "include")
LIB = os.path.join(CSRC, "libsvip.so")
DEBUG_LIB = os.path.join(CSRC, "libsvip_debug.so")
DEBUG_FLAGS = ["-DSVIP_DEBUG_BOUNDS", "-DSVIP_NVTX"]
SOURCES = ["svip.cu"]
HEADERS = sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cuh")) + \
    [os.path.join(INCLUDE, "svip.h")]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the SVIP CUDA library cannot be built")


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = DEBUG_LIB if debug else LIB
    if not force and not is_stale(lib):
        return lib
    tmp = lib + ".%d.tmp" % os.getpid()
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC, "-cudart", "static",
           "-o", tmp]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if debug:
        cmd += DEBUG_FLAGS + ["-ldl"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
