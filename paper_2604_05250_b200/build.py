"""Builds the CUDA library in-tree: csrc/*.cu -> libdualdiff.so (sm_100a only)."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdualdiff.so")
LIB_CHECK = os.path.join(HERE, "libdualdiff_check.so")      # the same sources with -DDD_BOUNDS_CHECK

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib=None) -> bool:
    lib = lib or LIB
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(HERE, "..", "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, extra_flags=()) -> str:
    if force or _stale():
        cmd = [_nvcc(), *NVCC_FLAGS, *extra_flags, "-o", LIB, *sources()]
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.run(cmd, check=True)
    return LIB


def build_check(force: bool = False, verbose: bool = False) -> str:
    """The bounds-checked build: every index the verification kernels form is compared with its
    extent and a violation goes to the health word (stand-in for a memory checker; the parity
    tests run a sample of their cases through it)."""
    if force or _stale(LIB_CHECK):
        cmd = [_nvcc(), *NVCC_FLAGS, "-DDD_BOUNDS_CHECK", "-o", LIB_CHECK, *sources()]
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.run(cmd, check=True)
    return LIB_CHECK


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose=True,
          extra_flags=["-Xptxas", "-v"] if "--ptxas" in sys.argv else [])
    print(LIB)
    if "--check" in sys.argv:
        print(build_check(force="--force" in sys.argv, verbose=True))
