"""Builds and runs the stand-alone probes (``csrc/probes``): the INT32 instruction rates the
integer epilogues depend on, the tcgen05 kind::i8 MMA issue rate, and the rates of the data paths of a
GEMM epilogue (TMEM loads, shared-memory byte stores and table loads).  All are stand-alone CUDA
programs; their output is what the ALU and INT8 peaks quoted for the kernels rest on.

    python -m paper_2101_01321_b200.probes [int|mma|epilogue]
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
PROBES = {"int": "int_issue_probe.cu", "mma": "mma_issue_probe.cu", "epilogue": "epilogue_path_probe.cu"}


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
