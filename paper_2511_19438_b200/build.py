"""Builds libgptq_b200.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libgptq_b200.so")
SOURCES = [os.path.join(CSRC, "gptq_b200.cu")]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--use_fast_math", "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
]


def _deps():
    out = list(SOURCES)
    for root in (CSRC, os.path.join(os.path.dirname(HERE), "include")):
        for f in os.listdir(root):
            if f.endswith((".cuh", ".h")):
                out.append(os.path.join(root, f))
    return out


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in _deps())


def _compile(out: str, extra, verbose: bool) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = out + f".{os.getpid()}.tmp"
    cmd = [nvcc] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + SOURCES
    subprocess.check_call(cmd)
    os.replace(tmp, out)
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not stale():
        return LIB
    extra = os.environ.get("GPTQ_NVCC_EXTRA", "").split()      # e.g. -DGPTQ_UMMA_MIN_TOKENS=17
    return _compile(LIB, extra, verbose)


TIMELINE_LIB = os.path.join(HERE, "libgptq_b200_timeline.so")


def build_timeline(force: bool = False) -> str:
    """The same library with the launch timeline compiled in (-DGPTQ_TIMELINE), as a file of its own."""
    if not force and os.path.exists(TIMELINE_LIB) and not any(os.path.getmtime(p) > os.path.getmtime(TIMELINE_LIB) for p in _deps()):
        return TIMELINE_LIB
    return _compile(TIMELINE_LIB, ["-DGPTQ_TIMELINE"], False)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
