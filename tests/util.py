"""Shared helpers of the test-suite (no arithmetic of the method)."""
import numpy as np

HP = dict(lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
STATE_NAMES = ("w", "m", "v", "d", "look")


def relerr(a, b):
    """max |a - b| / max(|a|, |b|), 0 where both are 0."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.maximum(np.abs(a), np.abs(b))
    with np.errstate(invalid="ignore", divide="ignore"):
        e = np.where(den > 0, np.abs(a - b) / den, 0.0)
    return float(e.max()) if e.size else 0.0


class DevicePtr:
    """Lets torch view library-owned device memory (float32 [rows, stride])."""

    def __init__(self, ptr, rows, stride):
        self.__cuda_array_interface__ = {
            "shape": (rows, stride), "typestr": "<f4", "data": (int(ptr), False),
            "version": 3, "strides": None}
