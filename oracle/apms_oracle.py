"""ctypes front end of the C oracle (test infrastructure only).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this.
State arrays are exposed as numpy views onto the oracle's own memory.
"""
from __future__ import annotations

import ctypes as C
from typing import Sequence

import numpy as np

from . import build as _build

ONEBIT, IDENTITY, TOPK = 0, 1, 2
VARIANT_MOMENTUM, VARIANT_GRADIENT = 0, 1
SCALE_L2, SCALE_L1_MEAN = 0, 1

_F = C.POINTER(C.c_float)
_U = C.POINTER(C.c_uint32)
_lib = None


def lib(path: str | None = None) -> C.CDLL:
    global _lib
    if path is not None:
        return _declare(C.CDLL(path))
    if _lib is None:
        _lib = _declare(C.CDLL(_build.build()))
    return _lib


def _declare(L: C.CDLL) -> C.CDLL:
    vp = C.c_void_p
    L.apms_oracle_create.restype = vp
    L.apms_oracle_create.argtypes = [C.c_int64, C.c_int, C.c_float, C.c_float, C.c_float,
                                     C.c_float, C.c_int64]
    L.apms_oracle_destroy.argtypes = [vp]
    L.apms_oracle_set_params.argtypes = [vp, _F]
    L.apms_oracle_set_lr.argtypes = [vp, C.c_float]
    for f in ("set_compressor", "set_scale_kind", "set_threads", "set_variant"):
        getattr(L, "apms_oracle_" + f).argtypes = [vp, C.c_int]
    L.apms_oracle_max_threads.restype = C.c_int
    for f in ("x", "m", "v", "server_err", "server_scales"):
        getattr(L, "apms_oracle_" + f).restype = _F
        getattr(L, "apms_oracle_" + f).argtypes = [vp]
    for f in ("worker_err", "worker_scales"):
        getattr(L, "apms_oracle_" + f).restype = _F
        getattr(L, "apms_oracle_" + f).argtypes = [vp, C.c_int]
    L.apms_oracle_worker_bits.restype = _U
    L.apms_oracle_worker_bits.argtypes = [vp, C.c_int]
    L.apms_oracle_server_bits.restype = _U
    L.apms_oracle_server_bits.argtypes = [vp]
    for f in ("warmup_step", "compressed_step"):
        getattr(L, "apms_oracle_" + f).restype = C.c_int
        getattr(L, "apms_oracle_" + f).argtypes = [vp, C.POINTER(_F)]
    L.apms_oracle_freeze_v.restype = C.c_int
    L.apms_oracle_freeze_v.argtypes = [vp]
    L.apms_oracle_t.restype = C.c_int
    L.apms_oracle_t.argtypes = [vp]
    L.apms_oracle_compress_1bit.argtypes = [_F, C.c_int64, C.c_int, _U, _F]
    L.apms_oracle_compress_topk.argtypes = [_F, C.c_int64, C.c_int64, _F, C.POINTER(C.c_uint8)]
    L.apms_oracle_topk_count.restype = C.c_int64
    L.apms_oracle_topk_count.argtypes = [C.c_double, C.c_int64]
    L.apms_oracle_set_topk_fraction.argtypes = [vp, C.c_double]
    L.apms_oracle_worker_selected.restype = C.POINTER(C.c_uint8)
    L.apms_oracle_worker_selected.argtypes = [vp, C.c_int]
    L.apms_oracle_server_selected.restype = C.POINTER(C.c_uint8)
    L.apms_oracle_server_selected.argtypes = [vp]
    L.apms_oracle_decompress_1bit.argtypes = [_U, C.c_float, C.c_int64, _F]
    return L


def _view(ptr, count, dtype):
    return np.ctypeslib.as_array(ptr, shape=(count,)).view(dtype)


def compress_1bit(z: np.ndarray, scale_kind: int = SCALE_L2, library: C.CDLL | None = None):
    """C[z] on one chunk: (sign words uint32[ceil(L/32)], scale float32)."""
    L = library or lib()
    z = np.ascontiguousarray(z, dtype=np.float32)
    bits = np.zeros((z.size + 31) // 32, dtype=np.uint32)
    scale = C.c_float(0.0)
    L.apms_oracle_compress_1bit(z.ctypes.data_as(_F), z.size, scale_kind,
                                bits.ctypes.data_as(_U), C.byref(scale))
    return bits, np.float32(scale.value)


def compress_topk(z: np.ndarray, K: int, library: C.CDLL | None = None):
    """Top-k C[z] on one chunk: (decompressed vector float32[L], mask of kept elements uint8[L])."""
    L = library or lib()
    z = np.ascontiguousarray(z, dtype=np.float32)
    q = np.empty(z.size, dtype=np.float32)
    sel = np.empty(z.size, dtype=np.uint8)
    L.apms_oracle_compress_topk(z.ctypes.data_as(_F), z.size, K, q.ctypes.data_as(_F),
                                sel.ctypes.data_as(C.POINTER(C.c_uint8)))
    return q, sel


def topk_count(frac: float, length: int, library: C.CDLL | None = None) -> int:
    return int((library or lib()).apms_oracle_topk_count(frac, length))


def decompress_1bit(bits: np.ndarray, scale, length: int, library: C.CDLL | None = None) -> np.ndarray:
    L = library or lib()
    bits = np.ascontiguousarray(bits, dtype=np.uint32)
    q = np.empty(length, dtype=np.float32)
    L.apms_oracle_decompress_1bit(bits.ctypes.data_as(_U), C.c_float(float(scale)), length,
                                  q.ctypes.data_as(_F))
    return q


class Oracle:
    """The optimizer state machine of Algorithm 1 on the CPU."""

    def __init__(self, d: int, n: int, beta1: float, beta2: float, eps: float, lr: float,
                 chunk: int, library: C.CDLL | None = None):
        self._L = library or lib()
        self._h = self._L.apms_oracle_create(d, n, beta1, beta2, eps, lr, chunk)
        if not self._h:
            raise ValueError("invalid oracle configuration")
        self.d, self.n, self.chunk = d, n, chunk
        self.C = (d + chunk - 1) // chunk
        self.W = (d + 31) // 32

    def close(self):
        if self._h:
            self._L.apms_oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    # configuration
    def set_params(self, x0: np.ndarray):
        x0 = np.ascontiguousarray(x0, dtype=np.float32)
        assert x0.size == self.d
        self._L.apms_oracle_set_params(self._h, x0.ctypes.data_as(_F))

    def set_lr(self, lr: float):
        self._L.apms_oracle_set_lr(self._h, lr)

    def set_compressor(self, kind: int):
        self._L.apms_oracle_set_compressor(self._h, kind)

    def set_topk_fraction(self, frac: float):
        self._L.apms_oracle_set_topk_fraction(self._h, frac)

    def worker_selected(self, i: int):
        return _view(self._L.apms_oracle_worker_selected(self._h, i), self.d, np.uint8)

    @property
    def server_selected(self):
        return _view(self._L.apms_oracle_server_selected(self._h), self.d, np.uint8)

    def set_variant(self, variant: int):
        self._L.apms_oracle_set_variant(self._h, variant)

    def set_scale_kind(self, kind: int):
        self._L.apms_oracle_set_scale_kind(self._h, kind)

    def set_threads(self, threads: int):
        self._L.apms_oracle_set_threads(self._h, threads)

    def max_threads(self) -> int:
        return int(self._L.apms_oracle_max_threads())

    # steps
    def _gptrs(self, grads: Sequence[np.ndarray]):
        assert len(grads) == self.n
        self._keep = [np.ascontiguousarray(g, dtype=np.float32) for g in grads]
        for g in self._keep:
            assert g.size == self.d
        return (_F * self.n)(*[g.ctypes.data_as(_F) for g in self._keep])

    def warmup_step(self, grads: Sequence[np.ndarray]):
        rc = self._L.apms_oracle_warmup_step(self._h, self._gptrs(grads))
        if rc:
            raise RuntimeError(f"oracle warmup_step: bad state ({rc})")

    def freeze_v(self):
        rc = self._L.apms_oracle_freeze_v(self._h)
        if rc:
            raise RuntimeError(f"oracle freeze_v: bad state ({rc})")

    def compressed_step(self, grads: Sequence[np.ndarray]):
        rc = self._L.apms_oracle_compressed_step(self._h, self._gptrs(grads))
        if rc:
            raise RuntimeError(f"oracle compressed_step: bad state ({rc})")

    # state views (live memory of the oracle; copy before the next step if needed)
    @property
    def t(self) -> int:
        return int(self._L.apms_oracle_t(self._h))

    @property
    def x(self):
        return _view(self._L.apms_oracle_x(self._h), self.d, np.float32)

    @property
    def m(self):
        return _view(self._L.apms_oracle_m(self._h), self.d, np.float32)

    @property
    def v(self):
        return _view(self._L.apms_oracle_v(self._h), self.d, np.float32)

    @property
    def server_err(self):
        return _view(self._L.apms_oracle_server_err(self._h), self.d, np.float32)

    @property
    def server_scales(self):
        return _view(self._L.apms_oracle_server_scales(self._h), self.C, np.float32)

    @property
    def server_bits(self):
        return _view(self._L.apms_oracle_server_bits(self._h), self.W, np.uint32)

    def worker_err(self, i: int):
        return _view(self._L.apms_oracle_worker_err(self._h, i), self.d, np.float32)

    def worker_scales(self, i: int):
        return _view(self._L.apms_oracle_worker_scales(self._h, i), self.C, np.float32)

    def worker_bits(self, i: int):
        return _view(self._L.apms_oracle_worker_bits(self._h, i), self.W, np.uint32)
