"""Builds libmcsd.so (the CUDA library behind the C ABI) in-tree with nvcc for sm_100a.

    python -m paper_2401_06706_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmcsd.so")
DEBUG_LIB = os.path.join(HERE, "libmcsd_debug.so")
SOURCES = [os.path.join(CSRC, "mcsd_api.cu")]
HEADERS = sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cuh")) + [os.path.join(ROOT, "include", "mcsd.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; libmcsd.so cannot be built")


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compile for sm_100a only; returns the path of the shared library.  debug_bounds: the checked
    build libmcsd_debug.so (-DMCSD_DEBUG_BOUNDS: reads of caller memory are checked, never trapped)."""
    lib = DEBUG_LIB if debug_bounds else LIB
    if not force and not is_stale(lib):
        return lib
    tmp = lib + f".{os.getpid()}.tmp"
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", tmp] + SOURCES
    if debug_bounds:
        cmd.insert(1, "-DMCSD_DEBUG_BOUNDS")
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
