"""CPU oracle for the COMP-AMS step (test infrastructure, not part of the product path).

`Oracle` wraps oracle/compams_oracle.cpp: Algorithm 2 (distributed COMP-AMS with error
feedback) with the Top-k and Block-Sign compressors of Definitions 1 and 2 and the AMSGrad
update of Algorithm 1, one plain loop per line of the algorithm. Only tests, the smoke check
and the benchmark's CPU-baseline leg may import this package; the CUDA library never does.
"""
from __future__ import annotations

import ctypes
from typing import Sequence

import numpy as np

from . import build as _build

TOPK = 0
BLOCKSIGN = 1
RANDK = 2

_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(_build.build())
        c = ctypes
        L.oracle_create.restype = c.c_void_p
        L.oracle_create.argtypes = [c.c_int32, c.c_int64, c.POINTER(c.c_int64), c.c_int32, c.c_int32, c.c_double,
                                    c.c_float, c.c_float, c.c_float, c.c_float]
        L.oracle_destroy.restype = None
        L.oracle_destroy.argtypes = [c.c_void_p]
        L.oracle_philox4x64_10.restype = None
        L.oracle_philox4x64_10.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p]
        L.oracle_randk_permute.restype = c.c_uint64
        L.oracle_randk_permute.argtypes = [c.c_uint64] * 6
        L.oracle_randk_block.restype = None
        L.oracle_randk_block.argtypes = [c.c_int64, c.c_int64, c.c_uint64, c.c_uint64, c.c_uint64, c.c_uint64, c.c_void_p]
        L.oracle_set_seed.restype = None
        L.oracle_set_seed.argtypes = [c.c_void_p, c.c_uint64, c.c_uint64]
        L.oracle_set_lr.restype = None
        L.oracle_set_lr.argtypes = [c.c_void_p, c.c_float]
        L.oracle_step.restype = c.c_int
        L.oracle_step.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p]
        L.oracle_buffer.restype = c.c_void_p
        L.oracle_buffer.argtypes = [c.c_void_p, c.c_int32, c.POINTER(c.c_int64)]
        L.oracle_kept_per_block.restype = c.c_int64
        L.oracle_kept_per_block.argtypes = [c.c_double, c.c_int64]
        L.oracle_topk_block.restype = None
        L.oracle_topk_block.argtypes = [c.c_void_p, c.c_int64, c.c_int64, c.c_void_p]
        L.oracle_blocksign_scale.restype = c.c_float
        L.oracle_blocksign_scale.argtypes = [c.c_void_p, c.c_int64]
        L.oracle_amsgrad.restype = None
        L.oracle_amsgrad.argtypes = [c.c_int64] + [c.c_void_p] * 5 + [c.c_float] * 4
        L.oracle_set_threads.restype = None
        L.oracle_set_threads.argtypes = [c.c_int32]
        L.oracle_max_threads.restype = c.c_int32
        L.oracle_max_threads.argtypes = []
        _lib = L
    return _lib


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def kept_per_block(k_ratio: float, d_b: int) -> int:
    """k for a block of size d_b: floor(k_ratio * d_b) clamped to [1, d_b]."""
    return int(lib().oracle_kept_per_block(float(k_ratio), int(d_b)))


def topk_keep_mask(x, k: int) -> np.ndarray:
    """Definition 1 on one block: boolean mask of the k kept coordinates (ties to the lower index)."""
    x = _f32(x)
    keep = np.zeros(x.size, dtype=np.uint8)
    lib().oracle_topk_block(x.ctypes.data, x.size, int(k), keep.ctypes.data)
    return keep.astype(bool)


def blocksign_scale(x) -> np.float32:
    """Definition 2 scale of one block: ||x||_1 / len(x), rounded once to fp32."""
    x = _f32(x)
    return np.float32(lib().oracle_blocksign_scale(x.ctypes.data, x.size))


def philox4x64_10(counter, key) -> np.ndarray:
    """One block of Philox4x64-10: counter (4 uint64), key (2 uint64) -> 4 uint64."""
    c = np.ascontiguousarray(counter, dtype=np.uint64)
    k = np.ascontiguousarray(key, dtype=np.uint64)
    out = np.zeros(4, dtype=np.uint64)
    lib().oracle_philox4x64_10(c.ctypes.data, k.ctypes.data, out.ctypes.data)
    return out


def randk_permute(m: int, r: int, seed: int, step: int, worker: int, block: int) -> int:
    """Image of r under the keyed permutation of {0..m-1} that Random-k draws its index sets from."""
    return int(lib().oracle_randk_permute(int(m), int(r), int(seed), int(step), int(worker), int(block)))


def randk_keep_mask(length: int, k: int, seed: int, step: int, worker: int, block: int) -> np.ndarray:
    """Random-k on one block: boolean mask of the k kept coordinates for (seed, step, worker, block)."""
    keep = np.zeros(int(length), dtype=np.uint8)
    lib().oracle_randk_block(int(length), int(k), int(seed), int(step), int(worker), int(block), keep.ctypes.data)
    return keep.astype(bool)


def amsgrad(g, m, v, vhat, theta, lr, beta1, beta2, eps) -> None:
    """Algorithm 1 update, in place on the fp32 arrays m, v, vhat, theta."""
    for a in (g, m, v, vhat, theta):
        assert a.dtype == np.float32 and a.flags.c_contiguous
    lib().oracle_amsgrad(g.size, g.ctypes.data, m.ctypes.data, v.ctypes.data, vhat.ctypes.data, theta.ctypes.data,
                         float(lr), float(beta1), float(beta2), float(eps))


def set_threads(t: int) -> None:
    lib().oracle_set_threads(int(t))


def max_threads() -> int:
    return int(lib().oracle_max_threads())


class Oracle:
    """State of Algorithm 2 on the CPU: E [n, d], m, v, vhat [d], all zero at construction."""

    _NAMES = {"E": 0, "m": 1, "v": 2, "vhat": 3, "gbar": 4, "C": 5, "scales": 6, "kept_idx": 7, "seg_off": 8}

    def __init__(self, n: int, d: int, block_offsets: Sequence[int], compressor: int, k_ratio: float = 1.0,
                 lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8):
        self.n, self.d = int(n), int(d)
        offs = np.ascontiguousarray(block_offsets, dtype=np.int64)
        self.M = offs.size - 1
        self.compressor = int(compressor)
        self._h = lib().oracle_create(self.n, self.d, offs.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), self.M,
                                      self.compressor, float(k_ratio), float(lr), float(beta1), float(beta2),
                                      float(eps))
        if not self._h:
            raise ValueError("oracle_create rejected the arguments")

    def step(self, G: np.ndarray, theta: np.ndarray) -> None:
        """One iteration of Algorithm 2. G: [n, d] fp32 gradients; theta: [d] fp32, updated in place."""
        assert G.dtype == np.float32 and G.flags.c_contiguous and G.shape == (self.n, self.d)
        assert theta.dtype == np.float32 and theta.flags.c_contiguous and theta.shape == (self.d,)
        rc = lib().oracle_step(self._h, G.ctypes.data, theta.ctypes.data)
        if rc != 0:
            raise RuntimeError("oracle_step failed")

    def set_seed(self, seed: int, steps_done: int = 0) -> None:
        """Random-k: the seed of the index sets and the number of iterations already done."""
        lib().oracle_set_seed(self._h, int(seed), int(steps_done))

    def set_lr(self, lr: float) -> None:
        """eta_t of the following steps (Algorithm 2 lets the learning rate vary with t)."""
        lib().oracle_set_lr(self._h, float(lr))

    def buffer(self, name: str) -> np.ndarray:
        """A view (not a copy) of an oracle buffer, valid until the next step or close()."""
        which = self._NAMES[name]
        cnt = ctypes.c_int64(0)
        p = lib().oracle_buffer(self._h, which, ctypes.byref(cnt))
        if cnt.value == 0:
            dt = np.int32 if name == "kept_idx" else np.int64 if name == "seg_off" else np.float32
            return np.zeros(0, dtype=dt)
        if name == "kept_idx":
            a = np.ctypeslib.as_array(ctypes.cast(p, ctypes.POINTER(ctypes.c_int32)), shape=(cnt.value,))
            return a.reshape(self.n, -1)
        if name == "seg_off":
            return np.ctypeslib.as_array(ctypes.cast(p, ctypes.POINTER(ctypes.c_int64)), shape=(cnt.value,))
        a = np.ctypeslib.as_array(ctypes.cast(p, ctypes.POINTER(ctypes.c_float)), shape=(cnt.value,))
        if name in ("E", "C"):
            return a.reshape(self.n, self.d)
        if name == "scales":
            return a.reshape(self.n, self.M)
        return a

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib().oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
