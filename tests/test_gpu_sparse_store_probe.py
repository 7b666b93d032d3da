"""What the layout of the EMA state d rests on: on this GPU a scattered store of a whole
32-byte sector is no dearer than a store of half of one (it is cheaper: the memory system
need not fetch the other half), and sparse reads are cheap next to sparse stores.  With
four replicas a coordinate's d entry is 16 bytes, so the owner kernel moves d in pairs
of coordinates.  The probe (tests/sparse_store_probe.cu) times the access forms on an
array larger than L2; run with ``-s`` to see the table."""
import ctypes
import os
import subprocess

import pytest

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "sparse_store_probe.cu")
LIB = os.path.join(HERE, "libsparse_store_probe.so")
FORMS = ["loop only", "read 16 B", "store 16 B", "store 32 B sector", "store 16 B, compacted",
         "store 32 B sector, compacted"]


def build():
    if not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(SRC):
        subprocess.run(["nvcc", "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
                        "-Xcompiler", "-fPIC", "-shared", "-o", LIB, SRC], check=True)
    return LIB


def test_whole_sector_stores_are_not_dearer_than_half_sector_stores():
    lib = ctypes.CDLL(build())
    n = 1 << 28                                   # 4 GB of 16-byte entries
    ms = (ctypes.c_float * 6)()
    assert lib.sparse_store_probe(ctypes.c_ulonglong(n), ctypes.c_double(0.05), ms) == 0
    ms = list(ms)
    print()
    for name, t in zip(FORMS, ms):
        print("  %-32s %7.3f ms   (+%.3f over the loop; %.1f M entries touched)"
              % (name, t, t - ms[0], 0.05 * n / 1e6))
    assert ms[3] <= 1.1 * ms[2]
    assert ms[5] <= 1.1 * ms[4]
    assert ms[1] - ms[0] <= ms[2] - ms[0]         # sparse reads cost no more than sparse stores
