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
SOURCES = [os.path.join(CSRC, f) for f in ("a2sgd.cu", "a2sgd_checked.cu", "a2sgd_noalloc.cu")]
DEPENDS = SOURCES + [os.path.join(CSRC, f) for f in ("a2sgd_kernels.cuh", "a2sgd_segments.cuh", "a2sgd_select.cuh",
                                                     "a2sgd_kernel_table.h", "a2sgd_debug_check.h")] \
    + [os.path.join(ROOT, "include", "a2sgd.h")]

COMPILE_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--ftz=false", "--prec-div=true", "--prec-sqrt=true",   # a flushed subnormal would change its sign group
    "-Xcompiler", "-fPIC",
]
LINK_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-Xcompiler", "-fPIC", "-cudart", "static"]


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
        # the translation units are compiled side by side (the production and the checked copy of
        # the kernels take about the same time), then linked; the library is replaced atomically
        from concurrent.futures import ThreadPoolExecutor
        objs = [f"{LIB}.{os.getpid()}.{i}.o" for i in range(len(SOURCES))]

        def compile_one(job):
            src, obj = job
            cmd = [nvcc()] + COMPILE_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", "-o", obj, src]
            subprocess.check_call(cmd)

        tmp = f"{LIB}.{os.getpid()}.tmp"
        try:
            with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:
                list(pool.map(compile_one, zip(SOURCES, objs)))
            subprocess.check_call([nvcc()] + LINK_FLAGS + ["-o", tmp] + objs)
            os.replace(tmp, LIB)
        finally:
            for f in objs + [tmp]:
                if os.path.exists(f):
                    os.remove(f)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
