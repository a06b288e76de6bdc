"""Builds libibert_b200.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
CSRC = PKG / "csrc"
LIB = PKG / "libibert_b200.so"
SOURCES = ["api.cu", "host_consts.cpp", "rowops.cu", "gemm_i8.cu", "gemm_splitk_i8.cu", "gemm_ln_i8.cu", "attention_i8.cu", "no_alloc.cu"]


def _sources():
    return [CSRC / s for s in SOURCES if (CSRC / s).exists()]


def _source_hash() -> str:
    """Hash of every source the library is built from (file times do not survive a copy of the tree)."""
    import hashlib
    h = hashlib.sha256()
    deps = sorted(list(CSRC.glob("*.cu")) + list(CSRC.glob("*.cuh")) + list(CSRC.glob("*.h")) +
                  list(CSRC.glob("*.cpp")) + [PKG.parent / "include" / "ibert.h", Path(__file__)])
    for d in deps:
        h.update(d.name.encode())
        h.update(d.read_bytes())
    return h.hexdigest()


HASH_FILE = PKG / "libibert_b200.so.srchash"


def _stale() -> bool:
    if not LIB.exists() or not HASH_FILE.exists():
        return True
    return HASH_FILE.read_text().strip() != _source_hash()


def build(force: bool = False, verbose: bool = False) -> Path:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
             "-Xcompiler", "-fPIC,-ffp-contract=off", "--fmad=false"]
    if verbose:
        flags += ["-Xptxas", "-v"]
    # one nvcc per translation unit, side by side, then one link
    obj_dir = PKG / "build" / f"obj{os.getpid()}"
    obj_dir.mkdir(parents=True, exist_ok=True)
    jobs = []
    for src in _sources():
        obj = obj_dir / (src.stem + ".o")
        jobs.append((obj, subprocess.Popen([nvcc, *flags, "-c", "-o", str(obj), str(src)])))
    failed = [str(o) for o, p in jobs if p.wait() != 0]
    if failed:
        raise subprocess.CalledProcessError(1, f"nvcc -c ({', '.join(failed)})")
    tmp = LIB.with_suffix(f".tmp{os.getpid()}.so")
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-cudart", "static",
                           "-o", str(tmp), *[str(o) for o, _ in jobs]])
    os.replace(tmp, LIB)
    for o, _ in jobs:
        o.unlink()
    obj_dir.rmdir()
    HASH_FILE.write_text(_source_hash() + "\n")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
