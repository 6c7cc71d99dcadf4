"""Compile the CUDA library in-tree with nvcc for sm_100a (``python -m paper_2403_10616_b200.build``)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdipaco.so")
SOURCES = ["dipaco.cu", "static_sync.cu"]
DEPENDS = ["dipaco.cu", "static_sync.cu", "kernels.cuh", "plan.hpp", "host_mode.inl",
           os.path.join("..", "..", "include", "dipaco.h")]


def nvcc_command(out, verbose=False):
    cmd = ["nvcc", "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xcompiler", "-fPIC,-O2,-Wall,-pthread", "-shared", "-cudart", "static",
           "-o", out]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    return cmd + [os.path.join(CSRC, s) for s in SOURCES]


def is_stale():
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in DEPENDS)


def build(force=False, verbose=False):
    """Build libdipaco.so if it is missing or older than its sources; returns its path."""
    if force or verbose or is_stale():
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(nvcc_command(tmp, verbose))
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
