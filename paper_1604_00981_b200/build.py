"""Compile libsgdb.so for sm_100a with nvcc, in-tree, beside the binding.

Usage:  python -m paper_1604_00981_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(_HERE), "include")
LIB = os.path.join(_HERE, "libsgdb.so")
SOURCES = [os.path.join(CSRC, "sgdb.cu")]
_DEPS = SOURCES + [os.path.join(CSRC, "sgdb_kernels.cuh"), os.path.join(CSRC, "sgdb_device.cuh"),
                   os.path.join(INCLUDE, "sgdb.h")]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; libsgdb needs the CUDA toolkit to build")


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > built for d in _DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Build the shared library if it is missing or older than its sources; return its path."""
    if not (force or is_stale()):
        return LIB
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = [
        nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
        "-shared", "-Xcompiler", "-fPIC", "-I", INCLUDE, "-o", tmp,
    ] + SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
