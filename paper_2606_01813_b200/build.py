"""Build step for the CUDA library: nvcc -> libcadd.so next to this file (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libcadd.so")
SOURCES = [os.path.join(CSRC, "cadd_api.cu"), os.path.join(CSRC, "cadd_static_scratch.cu")]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(_ROOT, "include", "cadd.h")]
    return max(os.path.getmtime(p) for p in paths)


def nvcc_command(verbose: bool = False) -> list:
    cmd = ["nvcc", "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
           "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(_ROOT, "include"), "-I", CSRC,
           "-o", LIB] + SOURCES
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    return cmd


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libcadd.so if it is missing or older than its sources; returns its path."""
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < _newest_source_mtime():
        subprocess.check_call(nvcc_command(verbose))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
