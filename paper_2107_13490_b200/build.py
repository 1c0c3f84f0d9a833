"""Builds libadapt_b200.so (CUDA kernels + C ABI) for sm_100a with nvcc, in-tree.

    python -m paper_2107_13490_b200.build [--force] [--check]

--check also builds libadapt_b200_check.so, the same library with every data-dependent table
index tested against its table's size (-DADAPT_CHECK_BOUNDS; see adapt_bounds_check_status).
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libadapt_b200.so")
CHECK_LIB = os.path.join(HERE, "libadapt_b200_check.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    # no FMA contraction anywhere: every fp32 step that decides an integer is one IEEE operation
    "-fmad=false",
    "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-ffp-contract=off",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        [os.path.join(os.path.dirname(HERE), "include", "adapt.h")]


def build(force: bool = False, verbose: bool = False, check: bool = False) -> str:
    """Builds the library (or, with check=True, its bounds-checking twin) if it is stale."""
    lib = CHECK_LIB if check else LIB
    stale = (not os.path.exists(lib)) or any(
        os.path.getmtime(d) > os.path.getmtime(lib) for d in _deps())
    if force or stale:
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = lib + ".tmp%d" % os.getpid()
        cmd = [nvcc] + NVCC_FLAGS + (["-DADAPT_CHECK_BOUNDS"] if check else []) + \
            (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + sources()
        subprocess.run(cmd, check=True)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--check" in sys.argv:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, check=True))
