"""Build the CUDA library in-tree: nvcc, sm_100a only.

    python -m paper_2010_16165_b200.build [--force] [--verbose]

Produces ``paper_2010_16165_b200/libfupruner.so`` (C ABI declared in include/fupruner.h).
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OUT = os.path.join(HERE, "libfupruner.so")
SOURCES = ["api.cu", "prep_kernels.cu", "mem_kernels.cu", "conv_simt.cu", "conv_tc.cu", "chain_tc.cu", "stem_pool.cu", "static_rank.cu"]


def lib_path():
    return OUT


def _newest_source():
    files = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    files.append(os.path.join(HERE, "..", "include", "fupruner.h"))
    return max(os.path.getmtime(f) for f in files)


def build(force=False, verbose=False):
    if not force and os.path.exists(OUT) and os.path.getmtime(OUT) >= _newest_source():
        return OUT
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-o", OUT]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    return OUT


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="--verbose" in sys.argv)
    print(OUT)
