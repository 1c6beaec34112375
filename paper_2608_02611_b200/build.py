"""Build the CUDA library in-tree:  python -m paper_2608_02611_b200.build

One translation unit (csrc/kb_host.cu) compiled by nvcc for sm_100a into
paper_2608_02611_b200/libkb.so, a plain C-ABI shared library (include/kb.h).
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libkb.so")
SOURCES = ["kb_host.cu"]
DEPS = ["kb_host.cu", "kb_common.cuh", "kb_screen.cuh", "kb_screen8.cuh", "kb_ring.cuh", "kb_screen64.cuh", "kb_adjudicate.cuh", "kb_select.cuh",
        os.path.join("..", "..", "include", "kb.h"), os.path.join("..", "..", "include", "kb_hooks.h")]

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-Wno-format-truncation", "-shared", "-ldl",
]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or stale():
        nvcc = os.environ.get("NVCC", "nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
              ["-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES]
        subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
