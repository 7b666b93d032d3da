"""Seeded synthetic inputs (initial weights, gradients) for tests and benches.

This module is the one piece both the CPU oracle's tests and the CUDA library's
tests draw from.  It holds none of the update's arithmetic: it only fills
arrays with reproducible pseudo-normal numbers, on the host (numpy) or on the
device (a small fill kernel), and the two fills agree bit for bit.

Recipe.  A stream is named by (seed, kind, step, stage, replica); its value at
coordinate c is a function of (stream, c) alone, so any slice of any stream can
be produced anywhere without producing the rest:

    key = mix(mix(mix(mix(seed + kind) + step) + stage) + replica)
    h   = mix(key + c)                              (mix = splitmix64 finaliser)
    s   = sum of the four 16-bit fields of h        (Irwin-Hall, n = 4)
    x   = float32(s - 131070) * float32(sigma / sqrt(1431655765))

The sum of four uniform 16-bit integers has mean 131070 and variance
4 * (65536^2 - 1) / 12 = 1431655765; it approximates a normal law with support
+-3.46 sigma.  Everything before the single fp32 multiply is integer-exact,
which is what makes host and device fills identical.
"""
from __future__ import annotations

import numpy as np

KIND_INIT = 1
KIND_GRAD = 2

_M64 = (1 << 64) - 1
IH_MEAN = 131070
IH_VAR = 1431655765.0


def _mix_int(x: int) -> int:
    x = (x + 0x9E3779B97F4A7C15) & _M64
    z = x
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, kind: int, step: int = 0, stage: int = 0,
               replica: int = 0) -> int:
    k = _mix_int((seed + kind) & _M64)
    k = _mix_int((k + step) & _M64)
    k = _mix_int((k + stage) & _M64)
    k = _mix_int((k + replica) & _M64)
    return k


def scale_f32(sigma: float) -> np.float32:
    return np.float32(sigma / np.sqrt(IH_VAR))


def normal_host(key: int, coord0: int, n: int, sigma: float) -> np.ndarray:
    """float32[n]: the stream ``key`` at coordinates coord0 .. coord0+n-1."""
    with np.errstate(over="ignore"):
        x = np.arange(coord0, coord0 + n, dtype=np.uint64) + np.uint64(key)
        x = x + np.uint64(0x9E3779B97F4A7C15)
        z = (x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        h = z ^ (z >> np.uint64(31))
    m = np.uint64(0xFFFF)
    s = ((h & m) + ((h >> np.uint64(16)) & m) + ((h >> np.uint64(32)) & m)
         + (h >> np.uint64(48))).astype(np.int64) - IH_MEAN
    return s.astype(np.float32) * scale_f32(sigma)


def init_weights_host(seed: int, stage: int, coord0: int, n: int,
                      sigma: float = 0.02) -> np.ndarray:
    """Initial weights of a stage (the same vector for every replica)."""
    return normal_host(stream_key(seed, KIND_INIT, 0, stage, 0), coord0, n, sigma)


def grads_host(seed: int, step: int, stage: int, R: int, coord0: int, n: int,
               sigma: float = 1e-3) -> np.ndarray:
    """float32[R, n]: gradients of step ``step`` for all replicas of a stage."""
    return np.stack([
        normal_host(stream_key(seed, KIND_GRAD, step, stage, i), coord0, n, sigma)
        for i in range(R)])


# ---- device fills (need the small CUDA library built from synth_fill.cu) -------

import ctypes as _ct
import os as _os
import shutil as _sh
import subprocess as _sp

_HERE = _os.path.dirname(_os.path.abspath(__file__))
_SRC = _os.path.join(_HERE, "synth_fill.cu")
_LIB = _os.path.join(_HERE, "libsynth_inputs.so")
_dev = None


def build(force: bool = False) -> str:
    stale = not _os.path.exists(_LIB) or _os.path.getmtime(_LIB) < _os.path.getmtime(_SRC)
    if force or stale:
        nvcc = _sh.which("nvcc") or "/usr/local/cuda/bin/nvcc"
        tmp = _LIB + ".tmp.%d" % _os.getpid()
        _sp.run([nvcc, "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
                 "-fmad=false", "-Xcompiler", "-fPIC", "-shared", "-o", tmp, _SRC], check=True)
        _os.replace(tmp, _LIB)
    return _LIB


def _devlib():
    global _dev
    if _dev is None:
        L = _ct.CDLL(build())
        L.synth_fill_normal.restype = _ct.c_int
        L.synth_fill_normal.argtypes = [_ct.c_void_p, _ct.c_uint64, _ct.c_uint64, _ct.c_uint64,
                                        _ct.c_float, _ct.c_void_p]
        _dev = L
    return _dev


def normal_device(dst, key: int, coord0: int, sigma: float) -> None:
    """Fill the 1-D CUDA float32 tensor ``dst`` with the stream ``key`` starting
    at coordinate ``coord0`` (same values as ``normal_host``)."""
    import torch
    assert dst.is_cuda and dst.dtype == torch.float32 and dst.is_contiguous()
    rc = _devlib().synth_fill_normal(dst.data_ptr(), dst.numel(), coord0, key,
                                     float(scale_f32(sigma)),
                                     torch.cuda.current_stream(dst.device).cuda_stream)
    if rc != 0:
        raise RuntimeError("synth_fill_normal: CUDA error %d" % rc)


def grads_device(dst, seed: int, step: int, stage: int, numel: int, sigma: float = 1e-3) -> None:
    """dst: CUDA float32 [R, stride] with stride >= numel; row i <- replica i's
    gradient of ``step``; padding columns are left untouched."""
    for i in range(dst.shape[0]):
        normal_device(dst[i, :numel], stream_key(seed, KIND_GRAD, step, stage, i), 0, sigma)
