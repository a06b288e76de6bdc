"""Builds and runs the two issue-rate probes (``csrc/probes``): the INT32 instruction rates the
integer epilogues depend on, and the tcgen05 kind::i8 MMA issue rate.  Both are stand-alone CUDA
programs; their output is what the ALU and INT8 peaks quoted for the kernels rest on.

    python -m paper_2101_01321_b200.probes [int|mma]
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
PROBES = {"int": "int_issue_probe.cu", "mma": "mma_issue_probe.cu"}


def build(name: str) -> Path:
    src = PKG / "csrc" / "probes" / PROBES[name]
    out_dir = PKG / "build"
    out_dir.mkdir(exist_ok=True)
    exe = out_dir / src.stem
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17",
                           "-o", str(exe), str(src)])
    return exe


def main(argv):
    names = argv or list(PROBES)
    for n in names:
        exe = build(n)
        print(f"== {PROBES[n]}", flush=True)
        subprocess.check_call([str(exe)])


if __name__ == "__main__":
    main(sys.argv[1:])
