"""Builds libqe.so (the C-ABI library) in-tree with nvcc for sm_100a.

    python -m paper_2609_23536_b200.build

The sources are compiled for compute_100a / sm_100a only; nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OUT = os.path.join(HERE, "libqe.so")
SOURCES = ["error.cpp", "contract.cpp", "kernels_hbm.cu", "gemm_sm100.cu", "layer_core.cu", "layer.cu", "layer_group.cu",
           "standalone.cu", "noalloc.cu"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", shutil.which("nvcc")):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


def _stale() -> bool:
    if not os.path.exists(OUT):
        return True
    t = os.path.getmtime(OUT)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "qe.h"), __file__]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return OUT
    srcs = [os.path.join(CSRC, s) for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]
    cmd = [
        _nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
        "-Xcompiler", "-fPIC,-Wall",
        # keep the static CUDA runtime private to this library (another runtime may already be loaded globally)
        "-Xlinker", "--exclude-libs,ALL", "-Xlinker", "-Bsymbolic", "-Xptxas", "-v" if verbose else "-O3",
        "-I", INCLUDE, "-I", CSRC, "-shared", "-o", OUT,
    ] + srcs
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed building libqe.so")
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
