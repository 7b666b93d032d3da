"""CPU oracle for the AsyncMesh per-step update -- TEST INFRASTRUCTURE ONLY.

This package wraps ``asyncmesh_oracle.c`` (plain single-threaded C, fp32, one
IEEE operation per written operation) with ctypes.  It exists so that the CUDA
library can be checked against an independent statement of the paper's update
equations (Section 2.3 Eq. "sparta", Section 3.1 Eq. "asparta", Section 3.2
Eq. "ema" and the corrected averaging, Section 2.2 look-ahead).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
it.  It imports nothing from the CUDA package and the CUDA package imports
nothing from here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "asyncmesh_oracle.c")
_LIB = os.path.join(_HERE, "libasyncmesh_oracle.so")

# The flags are part of the oracle's definition: no contraction into FMA, no
# value-changing optimisation, so every written operation rounds once.
CFLAGS = ["-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off",
          "-fno-fast-math", "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object next to its source."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < os.path.getmtime(_SRC))
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u32, u64, i32 = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int32
        dbl, vp = ctypes.c_double, ctypes.c_void_p
        L.am_oracle_create.restype = vp
        L.am_oracle_create.argtypes = [u32, u32, vp, vp, dbl, u32, dbl, dbl, dbl,
                                       dbl, dbl, dbl, u64, vp, u32]
        L.am_oracle_set_optimizer.restype = None
        L.am_oracle_set_optimizer.argtypes = [vp, u32, dbl]
        L.am_oracle_set_exchange.restype = None
        L.am_oracle_set_exchange.argtypes = [vp, u32]
        L.am_oracle_set_snapshot_storage.restype = None
        L.am_oracle_set_snapshot_storage.argtypes = [vp, u32]
        L.am_oracle_set_correction.restype = None
        L.am_oracle_set_correction.argtypes = [vp, u32]
        L.am_oracle_ema_variance.restype = ctypes.c_int
        L.am_oracle_ema_variance.argtypes = [vp, u32, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
        L.am_oracle_exchanged.restype = ctypes.c_float
        L.am_oracle_exchanged.argtypes = [u32, ctypes.c_float]
        L.am_oracle_destroy.restype = None
        L.am_oracle_destroy.argtypes = [vp]
        L.am_oracle_init_params.restype = ctypes.c_int
        L.am_oracle_init_params.argtypes = [vp, u32, i32, vp, u64]
        L.am_oracle_step_ex.restype = ctypes.c_int
        L.am_oracle_step_ex.argtypes = [vp, vp, dbl, dbl]
        L.am_oracle_row.restype = ctypes.POINTER(ctypes.c_float)
        L.am_oracle_row.argtypes = [vp, u32, ctypes.c_int, u32]
        L.am_oracle_lookahead.restype = ctypes.c_int
        L.am_oracle_lookahead.argtypes = [vp, u32, u32, vp]
        L.am_oracle_mean_params.restype = ctypes.c_int
        L.am_oracle_mean_params.argtypes = [vp, u32, vp]
        L.am_oracle_consensus_error.restype = dbl
        L.am_oracle_consensus_error.argtypes = [vp, u32]
        L.am_oracle_subset_mask.restype = ctypes.c_int
        L.am_oracle_subset_mask.argtypes = [vp, u32, u64, vp]
        L.am_oracle_step_count.restype = u64
        L.am_oracle_step_count.argtypes = [vp]
        L.am_oracle_philox4x32_10.restype = None
        L.am_oracle_philox4x32_10.argtypes = [vp, vp, vp]
        L.am_oracle_threshold.restype = u64
        L.am_oracle_threshold.argtypes = [dbl]
        L.am_oracle_selected.restype = ctypes.c_int
        L.am_oracle_selected.argtypes = [u64, u64, u32, u64, u64]
        _lib = L
    return _lib


def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> tuple:
    """One Philox-4x32-10 block (Salmon et al., SC'11)."""
    c = (ctypes.c_uint32 * 4)(*ctr)
    k = (ctypes.c_uint32 * 2)(*key)
    o = (ctypes.c_uint32 * 4)()
    lib().am_oracle_philox4x32_10(c, k, o)
    return tuple(int(x) for x in o)


EXCHANGE = {"fp32": 0, "bf16": 1, "fp8": 2}
CORRECTION = {"ema": 0, "eager": 1}


def exchanged(x: float, exchange: str = "bf16") -> float:
    """A snapshot value as the other replicas see it (bf16 / fp8: rounded to that format)."""
    return float(lib().am_oracle_exchanged(EXCHANGE[exchange], float(x)))


def threshold(p: float) -> int:
    return int(lib().am_oracle_threshold(float(p)))


def selected(seed: int, p: float, stage: int, step: int, mu: int) -> bool:
    return bool(lib().am_oracle_selected(seed, threshold(p), stage, step, mu))


WHICH = {"w": 0, "m": 1, "v": 2, "d": 3, "look": 4, "what": 5, "wprev": 6}


class Oracle:
    """R replicas x S stages of flat fp32 parameters, stepped on the CPU.

    ``numel[j]`` coordinates are held for stage j; ``coord_base[j]`` (default
    0) is the global index of the first one, which lets an instance stand for a
    slice of a larger stage.  ``ema_beta`` is the paper's lambda (weight of the
    new staleness sample in Eq. "ema").
    """

    def __init__(self, R: int, numel: Sequence[int], p: float, tau: int,
                 ema_beta: float, lr: float = 3e-4, beta1: float = 0.9,
                 beta2: float = 0.95, eps: float = 1e-8,
                 weight_decay: float = 0.1, seed: int = 0x5EED,
                 lookahead_delay: Optional[Sequence[int]] = None,
                 coord_base: Optional[Sequence[int]] = None, avg_interval: int = 1,
                 optimizer: str = "adamw", momentum_decay: float = 4e-3,
                 exchange: str = "fp32", correction: str = "ema",
                 snapshot: str = "own-fp32"):
        self.R, self.S, self.tau = int(R), len(numel), int(tau)
        self.numel = [int(n) for n in numel]
        self.p, self.seed = float(p), int(seed)
        ne = (ctypes.c_uint64 * self.S)(*self.numel)
        cb = (ctypes.c_uint64 * self.S)(*(coord_base or [0] * self.S))
        dl = None
        if lookahead_delay is not None:
            dl = (ctypes.c_uint32 * self.S)(*[int(x) for x in lookahead_delay])
        self._h = lib().am_oracle_create(
            self.R, self.S, ne, cb, float(p), self.tau, float(ema_beta),
            float(lr), float(beta1), float(beta2), float(eps),
            float(weight_decay), self.seed, dl, int(avg_interval))
        if not self._h:
            raise ValueError("oracle: invalid configuration or out of memory")
        lib().am_oracle_set_optimizer(self._h, {"adamw": 0, "nadamw": 1}[optimizer],
                                      float(momentum_decay))
        lib().am_oracle_set_exchange(self._h, EXCHANGE[exchange])
        lib().am_oracle_set_correction(self._h, CORRECTION[correction])
        # "own-fp32": a replica's staleness sample uses its own unrounded snapshot;
        # "as-exchanged": the snapshot exists only in the exchanged precision
        lib().am_oracle_set_snapshot_storage(self._h, {"own-fp32": 0, "as-exchanged": 1}[snapshot])

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib().am_oracle_destroy(self._h)
            self._h = None

    __del__ = close

    def init_params(self, stage: int, src: np.ndarray, replica: int = -1) -> None:
        a = np.ascontiguousarray(src, dtype=np.float32)
        rc = lib().am_oracle_init_params(self._h, stage, replica,
                                         a.ctypes.data, a.size)
        if rc != 0:
            raise ValueError("oracle: init_params rejected its arguments")

    def step(self, grads: Sequence[np.ndarray], ema_beta_t: float = -1.0,
             lr_t: float = -1.0) -> None:
        """grads[j]: float32 array of shape (R, numel[j])."""
        keep = []
        for j, g in enumerate(grads):
            a = np.ascontiguousarray(g, dtype=np.float32)
            if a.shape != (self.R, self.numel[j]):
                raise ValueError("oracle: grads[%d] has shape %r" % (j, a.shape))
            keep.append(a)
        ptrs = (ctypes.c_void_p * self.S)(*[a.ctypes.data for a in keep])
        rc = lib().am_oracle_step_ex(self._h, ptrs, float(ema_beta_t),
                                     float(lr_t))
        if rc != 0:
            raise RuntimeError("oracle: step failed")

    def row(self, stage: int, which: str, replica: int) -> np.ndarray:
        p = lib().am_oracle_row(self._h, stage, WHICH[which], replica)
        if not p:
            raise ValueError("oracle: bad row request")
        return np.ctypeslib.as_array(p, shape=(self.numel[stage],)).copy()

    def get(self, stage: int, which: str) -> np.ndarray:
        """All replicas of one state array: shape (R, numel[stage])."""
        return np.stack([self.row(stage, which, i) for i in range(self.R)])

    def lookahead(self, stage: int, delay: int) -> np.ndarray:
        """Look-ahead weights for any delay, shape (R, numel[stage])."""
        out = np.empty((self.R, self.numel[stage]), dtype=np.float32)
        if lib().am_oracle_lookahead(self._h, stage, int(delay), out.ctypes.data) != 0:
            raise ValueError("oracle: bad lookahead request")
        return out

    def mean_params(self, stage: int) -> np.ndarray:
        out = np.empty(self.numel[stage], dtype=np.float32)
        lib().am_oracle_mean_params(self._h, stage, out.ctypes.data)
        return out

    def consensus_error(self, stage: int) -> float:
        return float(lib().am_oracle_consensus_error(self._h, stage))

    def ema_variance(self, stage: int) -> tuple:
        """(mean, max) over the stage's coordinates of the across-replica variance of d."""
        mean, mx = ctypes.c_double(), ctypes.c_double()
        if lib().am_oracle_ema_variance(self._h, stage, ctypes.byref(mean), ctypes.byref(mx)) != 0:
            raise ValueError("oracle: bad ema_variance request")
        return float(mean.value), float(mx.value)

    def subset_mask(self, stage: int, step: int) -> np.ndarray:
        out = np.empty(self.numel[stage], dtype=np.uint8)
        lib().am_oracle_subset_mask(self._h, stage, step, out.ctypes.data)
        return out.astype(bool)

    @property
    def step_count(self) -> int:
        return int(lib().am_oracle_step_count(self._h))
