"""Builds and runs the tcgen05.mma issue microbenchmark (csrc/mma_issue_bench.cu).

    python -m paper_2506_01215_b200.mma_issue_bench            # build for sm_100a, run on cuda:0
    python -m paper_2506_01215_b200.mma_issue_bench --build    # build only (no GPU needed)

It is a stand-alone program beside the library: it times what one issuing
thread can feed the tensor pipe, the quantity the issue loops of the attention
and scan kernels are built around.
"""
from __future__ import annotations

import argparse
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "csrc", "mma_issue_bench.cu")
EXE = os.path.join(HERE, "mma_issue_bench.bin")


def build() -> str:
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-I", os.path.join(HERE, "csrc"), "-I", os.path.join(os.path.dirname(HERE), "include"),
           "-o", EXE, SRC, "-lcuda"]
    subprocess.check_call(cmd)
    return EXE


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--build", action="store_true", help="compile only")
    a = ap.parse_args()
    if a.build or not os.path.exists(EXE) or os.path.getmtime(EXE) < os.path.getmtime(SRC):
        build()
    if a.build:
        return 0
    return subprocess.call([EXE])


if __name__ == "__main__":
    sys.exit(main())
