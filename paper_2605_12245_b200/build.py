"""Build step for libsoar.so: nvcc cross-compiles csrc/soar.cu for sm_100a, in-tree.

Usage: ``python -m paper_2605_12245_b200.build [--force] [--verbose]``.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SOURCES = [os.path.join(HERE, "csrc", "soar.cu")]
HEADERS = [os.path.join(ROOT, "include", "soar.h")]
LIB = os.path.join(HERE, "libsoar.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared",
]


def nvcc_path() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: libsoar.so cannot be built")
    return cand


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile the CUDA library when it is missing or older than its sources."""
    if force or stale():
        tmp = LIB + f".tmp{os.getpid()}"
        cmd = [nvcc_path(), *NVCC_FLAGS, "-I", os.path.join(ROOT, "include")]
        if verbose:
            cmd += ["-Xptxas", "-v"]
        cmd += [*SOURCES, "-o", tmp]
        subprocess.check_call(cmd)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
