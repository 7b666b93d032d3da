"""Compile the CUDA sources of this package, in-tree, for sm_100a.

``python -m paper_2601_22442_b200.build`` (or ``build_all()``) runs nvcc on the
files under ``csrc/`` and leaves ``libasyncmesh.so`` next to this file.  nvcc
cross-compiles, so this works on a machine without a GPU.
"""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libasyncmesh.so")

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    # one rounding per written operation: no contraction into FMA, IEEE divide
    # and square root, no flush-to-zero
    "-fmad=false", "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "-Xcompiler", "-fPIC", "-shared",
]


def nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def _stale(target: str, sources) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def build_all(force: bool = False, verbose: bool = False) -> str:
    sources = [os.path.join(CSRC, f) for f in sorted(os.listdir(CSRC))]
    sources.append(os.path.join(os.path.dirname(HERE), "include", "asyncmesh.h"))
    if force or _stale(LIB, sources):
        tmp = LIB + ".tmp.%d" % os.getpid()
        cmd = [nvcc(), *NVCC_FLAGS, "-o", tmp, os.path.join(CSRC, "asyncmesh.cu")]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        subprocess.run(cmd, check=True)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build_all(force=True))
