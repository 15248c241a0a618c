"""Compile the CUDA library (csrc/boa.cu) into libboa.so next to this file, for sm_100a."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libboa.so")
SOURCES = ["boa.cu", "boa_build.cu"]
DEPS = ["boa.cu", "boa_build.cu", "boa_search.cuh", os.path.join("..", "..", "include", "boa.h")]


def nvcc_command(extra=()):
    return (["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
             "--shared", "-Xcompiler", "-fPIC", "-o", LIB]
            + list(extra) + [os.path.join(CSRC, s) for s in SOURCES])


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or is_stale():
        cmd = nvcc_command(["-Xptxas", "-v"] if verbose else [])
        subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
