"""Builds and runs the instruction-cost micro-benchmark (csrc/microbench/instr_cost.cu):

    python -m paper_2604_05650_b200.instr_cost

prints, for the B200 it runs on, the cycles per tcgen05.mma of the shapes the attention
kernel issues and per warp instruction of ex2, the conversions, fma and the warp maximum.
The figures in profiles/ and the split and organisation choices of the library rest on
them; the library itself does not use this program.
"""
from __future__ import annotations

import os
import subprocess
import sys

from . import build as _build

SRC = os.path.join(_build.CSRC, "microbench", "instr_cost.cu")
EXE = os.path.join(os.path.dirname(os.path.abspath(__file__)), "instr_cost.bin")


def build() -> str:
    if os.path.exists(EXE) and os.path.getmtime(EXE) >= os.path.getmtime(SRC):
        return EXE
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-I", _build.CSRC,
                    "-o", EXE, SRC], check=True)
    return EXE


if __name__ == "__main__":
    sys.exit(subprocess.run([build()]).returncode)
