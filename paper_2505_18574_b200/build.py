"""Build ``libi8ops.so`` (CUDA, sm_100a) in-tree beside this file with nvcc.

Run as ``python -m paper_2505_18574_b200.build`` or call :func:`build`.  nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libi8ops.so")
SOURCES = ["api.cu"]


def _newest_source_mtime() -> float:
    t = os.path.getmtime(os.path.join(os.path.dirname(HERE), "include", "i8ops.h"))
    for name in os.listdir(CSRC):
        if name.endswith((".cu", ".cuh", ".h")):
            t = max(t, os.path.getmtime(os.path.join(CSRC, name)))
    return t


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; return its path."""
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source_mtime():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-o", LIB]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    cmd += ["-lcudart"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
