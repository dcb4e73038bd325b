"""Builds libdass.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2405_01943_b200.build [--force] [--verbose] [--bounds-check]

--bounds-check builds libdass_check.so beside it: the same sources as ONE translation unit with -DDASS_BOUNDS_CHECK, in
which every global load and store of the library's kernels is tested against the buffers the call was given (an
outside access is skipped and counted, never performed).  It stands in for a memory sanitizer in the GPU tests.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
import tempfile

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libdass.so")
CHECK_LIB = os.path.join(PKG, "libdass_check.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(f) > t for f in _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
          ["-I", os.path.join(ROOT, "include"), "-I", CSRC] + sources() + ["-o", tmp]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libdass.so")
    os.replace(tmp, LIB)
    return LIB


def build_bounds_check(force: bool = False) -> str:
    """libdass_check.so: every source file included into one translation unit, compiled with -DDASS_BOUNDS_CHECK."""
    if not force and not is_stale(CHECK_LIB):
        return CHECK_LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = CHECK_LIB + f".tmp{os.getpid()}"
    with tempfile.TemporaryDirectory() as work:
        unity = os.path.join(work, "dass_unity.cu")
        with open(unity, "w") as f:
            for src in sources():
                f.write(f'#include "{src}"\n')
        cmd = [nvcc] + NVCC_FLAGS + ["-DDASS_BOUNDS_CHECK", "-I", os.path.join(ROOT, "include"), "-I", CSRC, unity, "-o", tmp]
        res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libdass_check.so")
    os.replace(tmp, CHECK_LIB)
    return CHECK_LIB


if __name__ == "__main__":
    if "--bounds-check" in sys.argv:
        print(build_bounds_check(force="--force" in sys.argv))
    else:
        print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
