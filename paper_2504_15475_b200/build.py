"""Compile libersd.so for sm_100a next to this file (nvcc cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SRC = [os.path.join(HERE, "csrc", "ersd.cu"), os.path.join(HERE, "csrc", "ersd_tree.cpp")]
DEPS = SRC + [os.path.join(HERE, "csrc", "ersd_math.cuh"), os.path.join(HERE, "csrc", "ersd_kernel.inc"), os.path.join(HERE, "csrc", "ersd_cluster.inc"), os.path.join(HERE, "csrc", "ersd_cluster_top.inc"), os.path.join(HERE, "csrc", "ersd_gsd.inc"), os.path.join(ROOT, "include", "ersd.h")]
LIB = os.path.join(HERE, "libersd.so")


def nvcc_command(out: str, extra=()):
    return ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
            "--shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"),
            "-I", os.path.join(HERE, "csrc"), *extra, "-o", out, *SRC]


def build(force: bool = False, verbose: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in DEPS)):
        return LIB
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = nvcc_command(tmp, ("-Xptxas", "-v") if verbose else ())
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
