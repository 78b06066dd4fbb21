"""Builds the CUDA library in-tree: ``python -m paper_2103_07454_b200.build`` (``--debug``: the
bounds-checked build, ``libeventgrad_debug.so``)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = [os.path.join(HERE, "csrc", "eventgrad.cu"), os.path.join(HERE, "csrc", "eg_norms_static.cu")]
LIB = os.path.join(HERE, "libeventgrad.so")
LIB_DEBUG = os.path.join(HERE, "libeventgrad_debug.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")

FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--fmad=false",            # every fused multiply-add of the path is written out
    "-Xcompiler", "-fPIC", "-shared", "-DEG_FUSED_VPT=1", "-ldl",
]


def sources():
    d = os.path.join(HERE, "csrc")
    return [os.path.join(d, f) for f in sorted(os.listdir(d))] + [
        os.path.join(HERE, "..", "include", "eventgrad.h")]


def _compile(lib: str, extra, force: bool, verbose: bool) -> str:
    newest = max(os.path.getmtime(p) for p in sources())
    if force or not os.path.exists(lib) or os.path.getmtime(lib) < newest:
        cmd = [NVCC] + FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + ["-o", lib] + SRC
        subprocess.run(cmd, check=True)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    return _compile(LIB, [], force, verbose)


def build_debug(force: bool = False, verbose: bool = False) -> str:
    """The bounds-checked build (-DEG_DEBUG): every index a kernel forms into a table is compared
    with the table's size first; a miss sets a bit of the context's error word instead of
    touching memory.  Load it with EG_LIBRARY=<path> in the environment."""
    return _compile(LIB_DEBUG, ["-DEG_DEBUG"], force, verbose)


if __name__ == "__main__":
    if "--debug" in sys.argv:
        print(build_debug(force="--force" in sys.argv, verbose="-v" in sys.argv))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
