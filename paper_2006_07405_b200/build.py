"""Builds liba2sgd.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2006_07405_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "liba2sgd.so")
SOURCES = [os.path.join(CSRC, "a2sgd.cu"), os.path.join(CSRC, "a2sgd_noalloc.cu")]
DEPENDS = SOURCES + [os.path.join(CSRC, "a2sgd_kernels.cuh"), os.path.join(ROOT, "include", "a2sgd.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--ftz=false", "--prec-div=true", "--prec-sqrt=true",   # a flushed subnormal would change its sign group
    "-shared", "-Xcompiler", "-fPIC", "-cudart", "static",
]


def nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in DEPENDS if os.path.exists(d))


def build(force: bool = False, verbose: bool = False) -> str:
    if force or is_stale():
        tmp = f"{LIB}.{os.getpid()}.tmp"
        cmd = [nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + SOURCES
        subprocess.check_call(cmd)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
