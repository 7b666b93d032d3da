"""ctypes binding of ``libasyncmesh.so``: same names as the C ABI, argument
marshalling only.  Every step of the update runs in the CUDA kernels behind the
library; PyTorch appears here only as the provider of device memory and of the
stream the work is issued on.  There is no CPU path: if the library is missing
or no CUDA device is usable, calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libasyncmesh.so")

OK = 0
ERR_INVALID_ARG, ERR_OOM, ERR_CUDA = -1, -2, -3
ERR_BAD_STATE, ERR_UNSUPPORTED, ERR_DEVICE_STATUS = -4, -5, -6
FLAG_SMALL_RING = 1
FLAG_DIRECT_KERNEL = 2
FLAG_PIPELINED_KERNEL = 4
FLAG_BF16_EXCHANGE = 16
FLAG_DENSE_RING = 32
FLAG_FP8_EXCHANGE = 64
FLAG_KEEP_PREVIOUS = 128
FLAG_OWNER_KERNEL = 256
FLAG_TRACK_CONSENSUS = 512
FLAG_RING_AS_EXCHANGED = 1024
STATE = {"w": 0, "m": 1, "v": 2, "d": 3, "look": 4}

ALLOC_FN = ctypes.CFUNCTYPE(ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t)
FREE_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_void_p)


class Config(ctypes.Structure):
    """Mirror of ``asyncmesh_config`` (include/asyncmesh.h)."""
    _fields_ = [
        ("R", ctypes.c_uint32), ("S", ctypes.c_uint32),
        ("stage_numel", ctypes.POINTER(ctypes.c_uint64)),
        ("p", ctypes.c_double),
        ("tau", ctypes.c_uint32), ("flags", ctypes.c_uint32),
        ("ema_beta", ctypes.c_double),
        ("lr", ctypes.c_double), ("beta1", ctypes.c_double), ("beta2", ctypes.c_double),
        ("eps", ctypes.c_double), ("weight_decay", ctypes.c_double),
        ("seed", ctypes.c_uint64),
        ("lookahead_delay", ctypes.POINTER(ctypes.c_uint32)),
        ("device", ctypes.c_int32), ("avg_interval", ctypes.c_int32),
        ("stream", ctypes.c_void_p),
        ("alloc", ALLOC_FN), ("free", FREE_FN), ("alloc_ctx", ctypes.c_void_p),
        ("optimizer", ctypes.c_uint32), ("correction", ctypes.c_uint32),
        ("momentum_decay", ctypes.c_double),
        ("coord_base", ctypes.POINTER(ctypes.c_uint64)),
    ]


class AsyncMeshError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("asyncmesh error %d: %s" % (code, message))
        self.code = code


_lib: Optional[ctypes.CDLL] = None

# every symbol include/asyncmesh.h declares: name -> (restype, argtypes)
_vp, _u32, _u64, _i32, _int = (ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64,
                               ctypes.c_int32, ctypes.c_int)
SIGNATURES = {
    "asyncmesh_create": (_int, [ctypes.POINTER(Config), ctypes.POINTER(_vp)]),
    "asyncmesh_destroy": (_int, [_vp]),
    "asyncmesh_init_params": (_int, [_vp, _u32, _i32, _vp, _u64, _int]),
    "asyncmesh_row_stride": (_int, [_vp, _u32, ctypes.POINTER(_u64)]),
    "asyncmesh_step": (_int, [_vp, ctypes.POINTER(_vp)]),
    "asyncmesh_step_ex": (_int, [_vp, ctypes.POINTER(_vp), ctypes.c_double, ctypes.c_double]),
    "asyncmesh_step_host": (_int, [_vp, ctypes.POINTER(_vp)]),
    "asyncmesh_step_host_ex": (_int, [_vp, ctypes.POINTER(_vp), ctypes.c_double, ctypes.c_double]),
    "asyncmesh_kernel_name": (_int, [_vp, ctypes.c_char_p, ctypes.c_size_t]),
    "asyncmesh_lookahead_weights": (_int, [_vp, _u32, _u32, ctypes.POINTER(_vp),
                                           ctypes.POINTER(_u64)]),
    "asyncmesh_read_params": (_int, [_vp, _u32, _i32, _vp, _u64, _int]),
    "asyncmesh_read_state": (_int, [_vp, _u32, _int, _i32, _vp, _u64, _int]),
    "asyncmesh_read_state_range": (_int, [_vp, _u32, _int, _i32, _u64, _u64, _vp, _int]),
    "asyncmesh_subset_mask": (_int, [_vp, _u32, _u64, _vp]),
    "asyncmesh_consensus_error": (_int, [_vp, _u32, ctypes.POINTER(ctypes.c_double)]),
    "asyncmesh_ema_variance": (_int, [_vp, _u32, ctypes.POINTER(ctypes.c_double),
                                      ctypes.POINTER(ctypes.c_double)]),
    "asyncmesh_consensus_error_noalloc": (_int, [_int, _vp, _vp, _u32, _u64, _u64,
                                                 ctypes.POINTER(ctypes.c_double)]),
    "asyncmesh_step_count": (_int, [_vp, ctypes.POINTER(_u64)]),
    "asyncmesh_min_bytes_last_step": (_int, [_vp, ctypes.POINTER(_u64)]),
    "asyncmesh_status": (_int, [_vp]),
    "asyncmesh_debug_philox": (_int, [_int, _vp, _vp, _vp, _u64]),
    "asyncmesh_last_error": (ctypes.c_char_p, []),
}


def load() -> ctypes.CDLL:
    """Load the CUDA library (building it is ``build.build_all``'s job)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "%s is missing: run `python -m paper_2601_22442_b200.build` "
                "(there is no fallback path)" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != OK:
        raise AsyncMeshError(rc, load().asyncmesh_last_error().decode())


def asyncmesh_last_error() -> str:
    return load().asyncmesh_last_error().decode()


class TorchAllocator:
    """Device memory for the library, taken from PyTorch's caching allocator."""

    def __init__(self, device: int):
        import torch
        self._torch = torch
        self._device = torch.device("cuda", device)
        self._live: Dict[int, object] = {}
        self.alloc_cb = ALLOC_FN(self._alloc)
        self.free_cb = FREE_FN(self._free)
        self.bytes_live = 0
        self.fail_after_bytes: Optional[int] = None   # tests: simulate exhaustion

    def _alloc(self, _ctx, nbytes):
        try:
            if self.fail_after_bytes is not None and self.bytes_live + nbytes > self.fail_after_bytes:
                return None
            t = self._torch.empty(int(nbytes), dtype=self._torch.uint8, device=self._device)
        except Exception:   # out of memory: report NULL, the library cleans up
            return None
        self._live[t.data_ptr()] = t
        self.bytes_live += int(nbytes)
        return t.data_ptr()

    def _free(self, _ctx, ptr):
        t = self._live.pop(int(ptr), None)
        if t is not None:
            self.bytes_live -= t.numel()


class AsyncMesh:
    """Handle on R replicas x S stages held on one GPU.

    The methods are the C calls with the ``asyncmesh_`` prefix dropped; module
    level functions with the full names are provided below.
    """

    def __init__(self, R: int, stage_numel: Sequence[int], p: float, tau: int,
                 ema_beta: float, lr: float = 3e-4, beta1: float = 0.9,
                 beta2: float = 0.95, eps: float = 1e-8, weight_decay: float = 0.1,
                 seed: int = 0x5EED, lookahead_delay: Optional[Sequence[int]] = None,
                 device: int = 0, stream: Optional[int] = None,
                 allocator: Optional[TorchAllocator] = None,
                 use_torch_allocator: bool = True, flags: int = 0, avg_interval: int = 1,
                 optimizer: str = "adamw", momentum_decay: float = 4e-3,
                 correction: str = "ema", coord_base: Optional[Sequence[int]] = None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("asyncmesh needs a CUDA device; there is no CPU path")
        self._h = _vp()
        self.R, self.S, self.tau = int(R), len(stage_numel), int(tau)
        self.numel = [int(n) for n in stage_numel]
        self.device = int(device)
        self._torch = torch
        if stream is None:
            stream = torch.cuda.current_stream(self.device).cuda_stream
        self.allocator = allocator
        if self.allocator is None and use_torch_allocator:
            self.allocator = TorchAllocator(self.device)
        ne = (ctypes.c_uint64 * self.S)(*self.numel)
        dl = None
        if lookahead_delay is not None:
            dl = (ctypes.c_uint32 * self.S)(*[int(x) for x in lookahead_delay])
        cfg = Config()
        cfg.R, cfg.S = self.R, self.S
        cfg.stage_numel = ctypes.cast(ne, ctypes.POINTER(ctypes.c_uint64))
        cfg.p, cfg.tau, cfg.flags, cfg.ema_beta = float(p), self.tau, int(flags), float(ema_beta)
        cfg.lr, cfg.beta1, cfg.beta2 = float(lr), float(beta1), float(beta2)
        cfg.eps, cfg.weight_decay, cfg.seed = float(eps), float(weight_decay), int(seed)
        if dl is not None:
            cfg.lookahead_delay = ctypes.cast(dl, ctypes.POINTER(ctypes.c_uint32))
        cfg.device, cfg.avg_interval, cfg.stream = self.device, int(avg_interval), stream
        cfg.optimizer = {"adamw": 0, "nadamw": 1}[optimizer]
        cfg.correction = {"ema": 0, "eager": 1}[correction]
        if coord_base is not None:
            self._base = (ctypes.c_uint64 * self.S)(*[int(b) for b in coord_base])
            cfg.coord_base = self._base
        cfg.momentum_decay = float(momentum_decay)
        if self.allocator is not None:
            cfg.alloc, cfg.free = self.allocator.alloc_cb, self.allocator.free_cb
        h = _vp()
        _check(load().asyncmesh_create(ctypes.byref(cfg), ctypes.byref(h)))
        self._h = h
        self.delay = list(lookahead_delay) if lookahead_delay is not None else \
            [self.S - 1 - s for s in range(self.S)]
        self.stride = [self.row_stride(s) for s in range(self.S)]

    # -- life cycle ------------------------------------------------------------
    def destroy(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            load().asyncmesh_destroy(self._h)
            self._h = _vp()

    close = destroy

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.destroy()

    # -- parameters in ----------------------------------------------------------
    def init_params(self, stage: int, src, replica: int = -1) -> None:
        """src: numpy float32 array (host) or a CUDA float32 torch tensor."""
        if isinstance(src, np.ndarray):
            a = np.ascontiguousarray(src, dtype=np.float32)
            _check(load().asyncmesh_init_params(self._h, stage, replica, a.ctypes.data, a.size, 0))
        else:
            t = src.contiguous()
            assert t.is_cuda and t.dtype == self._torch.float32
            _check(load().asyncmesh_init_params(self._h, stage, replica, t.data_ptr(), t.numel(), 1))

    def row_stride(self, stage: int) -> int:
        out = _u64()
        _check(load().asyncmesh_row_stride(self._h, stage, ctypes.byref(out)))
        return int(out.value)

    def empty_grads(self) -> List["object"]:
        """Zeroed device gradient buffers of the right shape: [R, row_stride_j]."""
        dev = self._torch.device("cuda", self.device)
        return [self._torch.zeros((self.R, self.stride[s]), dtype=self._torch.float32, device=dev)
                for s in range(self.S)]

    # -- the step ----------------------------------------------------------------
    def _ptrs(self, bufs) -> "ctypes.Array":
        if len(bufs) != self.S:
            raise ValueError("need one gradient buffer per stage")
        return (_vp * self.S)(*[int(b) if isinstance(b, int) else b.data_ptr() for b in bufs])

    def step(self, grads, ema_beta_t: float = -1.0, lr_t: float = -1.0) -> None:
        """grads[j]: CUDA float32 tensor [R, row_stride_j] (or its address)."""
        ptrs = self._ptrs(grads)
        if ema_beta_t < 0 and lr_t < 0:
            _check(load().asyncmesh_step(self._h, ptrs))
        else:
            _check(load().asyncmesh_step_ex(self._h, ptrs, float(ema_beta_t), float(lr_t)))

    def step_host(self, grads_host, ema_beta_t: float = -1.0, lr_t: float = -1.0) -> None:
        """grads_host[j]: host float32 [R, numel_j], contiguous (numpy array or
        pinned CPU torch tensor)."""
        ptrs = []
        for j, g in enumerate(grads_host):
            if isinstance(g, np.ndarray):
                assert g.dtype == np.float32 and g.flags.c_contiguous
                assert g.size == self.R * self.numel[j]
                ptrs.append(g.ctypes.data)
            else:
                assert (not g.is_cuda) and g.is_contiguous() and g.numel() == self.R * self.numel[j]
                ptrs.append(g.data_ptr())
        if ema_beta_t < 0 and lr_t < 0:
            _check(load().asyncmesh_step_host(self._h, (_vp * self.S)(*ptrs)))
        else:
            _check(load().asyncmesh_step_host_ex(self._h, (_vp * self.S)(*ptrs), float(ema_beta_t),
                                                 float(lr_t)))

    # -- results out ---------------------------------------------------------------
    def lookahead_weights(self, stage: int, delay: int):
        """(device address, row stride in floats) of the look-ahead weights."""
        ptr, stride = _vp(), _u64()
        _check(load().asyncmesh_lookahead_weights(self._h, stage, delay, ctypes.byref(ptr),
                                                  ctypes.byref(stride)))
        return int(ptr.value), int(stride.value)

    def read_params(self, stage: int, replica: int = -1, out=None) -> np.ndarray:
        n = self.numel[stage]
        if out is not None and not isinstance(out, np.ndarray):
            _check(load().asyncmesh_read_params(self._h, stage, replica, out.data_ptr(), n, 1))
            return out
        dst = np.empty(n, dtype=np.float32) if out is None else out
        _check(load().asyncmesh_read_params(self._h, stage, replica, dst.ctypes.data, n, 0))
        return dst

    def read_state(self, stage: int, which: str, replica: int) -> np.ndarray:
        n = self.numel[stage]
        dst = np.empty(n, dtype=np.float32)
        _check(load().asyncmesh_read_state(self._h, stage, STATE[which], replica,
                                           dst.ctypes.data, n, 0))
        return dst

    def read_state_range(self, stage: int, which: str, replica: int, first: int,
                         count: int) -> np.ndarray:
        dst = np.empty(count, dtype=np.float32)
        _check(load().asyncmesh_read_state_range(self._h, stage, STATE[which], replica, first,
                                                 count, dst.ctypes.data, 0))
        return dst

    def get_range(self, stage: int, which: str, first: int, count: int) -> np.ndarray:
        """All replicas of one state array on a coordinate range: [R, count]."""
        return np.stack([self.read_state_range(stage, which, i, first, count)
                         for i in range(self.R)])

    def get(self, stage: int, which: str) -> np.ndarray:
        """All replicas of one state array: [R, numel[stage]]."""
        return np.stack([self.read_state(stage, which, i) for i in range(self.R)])

    def subset_mask(self, stage: int, step: int) -> np.ndarray:
        n = self.numel[stage]
        bm = np.zeros((n + 7) // 8, dtype=np.uint8)
        _check(load().asyncmesh_subset_mask(self._h, stage, step, bm.ctypes.data))
        return np.unpackbits(bm, bitorder="little")[:n].astype(bool)

    def consensus_error(self, stage: int) -> float:
        out = ctypes.c_double()
        _check(load().asyncmesh_consensus_error(self._h, stage, ctypes.byref(out)))
        return float(out.value)

    def ema_variance(self, stage: int) -> tuple:
        """(mean, max) over the stage's coordinates of the across-replica variance of d."""
        mean, mx = ctypes.c_double(), ctypes.c_double()
        _check(load().asyncmesh_ema_variance(self._h, stage, ctypes.byref(mean), ctypes.byref(mx)))
        return float(mean.value), float(mx.value)

    @property
    def step_count(self) -> int:
        out = _u64()
        _check(load().asyncmesh_step_count(self._h, ctypes.byref(out)))
        return int(out.value)

    def min_bytes_last_step(self) -> int:
        out = _u64()
        _check(load().asyncmesh_min_bytes_last_step(self._h, ctypes.byref(out)))
        return int(out.value)

    def status(self) -> None:
        _check(load().asyncmesh_status(self._h))

    def kernel_name(self) -> str:
        buf = ctypes.create_string_buffer(128)
        _check(load().asyncmesh_kernel_name(self._h, buf, 128))
        return buf.value.decode()


# ---- the C names, as functions ---------------------------------------------------

def asyncmesh_create(R, S, stage_numel, p, tau, ema_beta, **kw) -> AsyncMesh:
    if len(stage_numel) != S:
        raise ValueError("S does not match len(stage_numel)")
    return AsyncMesh(R, stage_numel, p, tau, ema_beta, **kw)


def asyncmesh_destroy(h: AsyncMesh) -> None:
    h.destroy()


def asyncmesh_init_params(h: AsyncMesh, stage, replica, src) -> None:
    h.init_params(stage, src, replica)


def asyncmesh_step(h: AsyncMesh, grads) -> None:
    h.step(grads)


def asyncmesh_step_ex(h: AsyncMesh, grads, ema_beta_t, lr_t) -> None:
    h.step(grads, ema_beta_t, lr_t)


def asyncmesh_step_host(h: AsyncMesh, grads_host) -> None:
    h.step_host(grads_host)


def asyncmesh_step_host_ex(h: AsyncMesh, grads_host, ema_beta_t, lr_t) -> None:
    h.step_host(grads_host, ema_beta_t, lr_t)


def asyncmesh_kernel_name(h: AsyncMesh) -> str:
    return h.kernel_name()


def asyncmesh_lookahead_weights(h: AsyncMesh, stage, delay):
    return h.lookahead_weights(stage, delay)


def asyncmesh_read_params(h: AsyncMesh, stage, replica=-1, out=None):
    return h.read_params(stage, replica, out)


def asyncmesh_read_state(h: AsyncMesh, stage, which, replica):
    return h.read_state(stage, which, replica)


def asyncmesh_read_state_range(h: AsyncMesh, stage, which, replica, first, count):
    return h.read_state_range(stage, which, replica, first, count)


def asyncmesh_subset_mask(h: AsyncMesh, stage, step):
    return h.subset_mask(stage, step)


def asyncmesh_ema_variance(h: AsyncMesh, stage):
    return h.ema_variance(stage)


def asyncmesh_consensus_error(h: AsyncMesh, stage):
    return h.consensus_error(stage)


def asyncmesh_consensus_error_noalloc(w_device: int, R: int, n: int, row_stride: int,
                                      device: int = 0, stream: int = 0) -> float:
    """Consensus error of the rows at device address ``w_device`` through the entry
    point that allocates nothing (its scratch is a fixed array inside the library,
    good for n <= 2**28).  For callers that must not trigger an allocation."""
    out = ctypes.c_double()
    _check(load().asyncmesh_consensus_error_noalloc(device, stream, w_device, R, n, row_stride,
                                                    ctypes.byref(out)))
    return float(out.value)


def asyncmesh_debug_philox(ctr: np.ndarray, key: np.ndarray, device: int = 0) -> np.ndarray:
    c = np.ascontiguousarray(ctr, dtype=np.uint32).reshape(-1, 4)
    k = np.ascontiguousarray(key, dtype=np.uint32).reshape(-1, 2)
    assert c.shape[0] == k.shape[0]
    out = np.empty_like(c)
    _check(load().asyncmesh_debug_philox(device, c.ctypes.data, k.ctypes.data,
                                         out.ctypes.data, c.shape[0]))
    return out
