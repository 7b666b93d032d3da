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

OBJ = os.path.join(HERE, "build")      # object files of the last build

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    # one rounding per written operation: no contraction into FMA, IEEE divide
    # and square root, no flush-to-zero
    "-fmad=false", "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "-Xcompiler", "-fPIC", "-Xfatbin", "-compress-all",
]

# translation units: the C ABI with its small kernels, and the step-kernel
# instantiations in twelve parts that compile side by side
UNITS = [("asyncmesh", "asyncmesh.cu", []),
         *[("step_kernels_%d" % k, "step_kernels.cu", ["-DAM_PART=%d" % k]) for k in range(12)]]


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


def build_all(force: bool = False, verbose: bool = False, extra_flags=(), lib: str = LIB) -> str:
    sources = [os.path.join(CSRC, f) for f in sorted(os.listdir(CSRC))]
    sources.append(os.path.join(os.path.dirname(HERE), "include", "asyncmesh.h"))
    if force or _stale(lib, sources):
        os.makedirs(OBJ, exist_ok=True)
        tag = "%d" % os.getpid()
        jobs = []
        for name, src, defs in UNITS:
            obj = os.path.join(OBJ, "%s.%s.o" % (name, tag))
            cmd = [nvcc(), *NVCC_FLAGS, *defs, *extra_flags, "-c", "-o", obj, os.path.join(CSRC, src)]
            if verbose:
                cmd[1:1] = ["-Xptxas", "-v"]
            jobs.append((obj, cmd, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT,
                                                    text=True)))
        objs, failed = [], []
        for obj, cmd, proc in jobs:
            out, _ = proc.communicate()
            if verbose or proc.returncode != 0:
                print(out, end="")
            if proc.returncode != 0:
                failed.append(" ".join(cmd))
            objs.append(obj)
        try:
            if failed:
                raise RuntimeError("nvcc failed: " + failed[0])
            tmp = lib + ".tmp." + tag
            subprocess.run([nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp, *objs],
                           check=True)
            os.replace(tmp, lib)
        finally:
            for obj in objs:
                if os.path.exists(obj):
                    os.remove(obj)
    return lib


if __name__ == "__main__":
    print(build_all(force=True))
