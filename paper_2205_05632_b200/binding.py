"""ctypes binding of the COMP-AMS C ABI (include/compams.h).

Argument marshalling only: every step of the optimizer iteration runs inside the CUDA library.
PyTorch supplies device memory and the CUDA stream. If the compiled library is missing the
first call raises CompAMSError; there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

TOPK = 0
BLOCKSIGN = 1
RANDK = 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libcompams.so"

BUFFERS = {
    "E": 0, "m": 1, "v": 2, "vhat": 3, "gbar": 4, "topk_idx": 5, "topk_val": 6, "topk_seg_offsets": 7,
    "sign_bits": 8, "sign_word_offsets": 9, "scales": 10, "status": 11,
}
_BUFFER_DTYPES = {
    "E": torch.float32, "m": torch.float32, "v": torch.float32, "vhat": torch.float32, "gbar": torch.float32,
    "topk_idx": torch.int32, "topk_val": torch.float32, "topk_seg_offsets": torch.int64,
    "sign_bits": torch.int32, "sign_word_offsets": torch.int64, "scales": torch.float32, "status": torch.int32,
}
_TYPESTR = {torch.float32: "<f4", torch.int32: "<i4", torch.int64: "<i8"}

KERNELS = {
    "dense_mean_amsgrad": 0, "bs_sweep": 1, "bs_apply": 2, "bs_materialize": 3, "topk_sweep": 4, "topk_dense": 5,
    "topk_materialize": 6, "randk_emit": 7, "topk_scatter": 9, "amsgrad": 10, "topk_small": 11,
    "topk_select": 12, "bs_scales": 13,
}


class CompAMSError(RuntimeError):
    pass


def library_path() -> str:
    return os.path.join(_HERE, _LIB_NAME)


_lib: Optional[ctypes.CDLL] = None


def load_library() -> ctypes.CDLL:
    """Load libcompams.so (built in-tree by paper_2205_05632_b200.build) and declare its symbols."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise CompAMSError(
            "CUDA library %s not found: build it with `python -m paper_2205_05632_b200.build` "
            "(there is no CPU fallback)" % path)
    L = ctypes.CDLL(path)
    c = ctypes
    H = c.c_void_p
    L.compams_create.restype = c.c_int
    L.compams_create.argtypes = [c.POINTER(H), c.c_int32, c.c_int64, c.POINTER(c.c_int64), c.c_int32, c.c_int32,
                                 c.c_double, c.c_float, c.c_float, c.c_float, c.c_float]
    L.compams_step.restype = c.c_int
    L.compams_step.argtypes = [H, c.c_void_p, c.c_void_p]
    L.compams_step_bf16.restype = c.c_int
    L.compams_step_bf16.argtypes = [H, c.c_void_p, c.c_void_p]
    L.compams_compress_bf16.restype = c.c_int
    L.compams_compress_bf16.argtypes = [H, c.c_void_p]
    L.compams_step_host.restype = c.c_int
    L.compams_step_host.argtypes = [H, c.c_void_p, c.c_void_p]
    L.compams_create_sharded.restype = c.c_int
    L.compams_create_sharded.argtypes = [c.POINTER(H), c.c_int32, c.c_int32, c.c_int32, c.c_int64, c.POINTER(c.c_int64),
                                         c.c_int32, c.c_int32, c.c_double, c.c_float, c.c_float, c.c_float, c.c_float]
    L.compams_workspace_bytes.restype = c.c_int
    L.compams_workspace_bytes.argtypes = [c.POINTER(c.c_size_t), c.c_int32, c.c_int32, c.c_int64, c.POINTER(c.c_int64),
                                          c.c_int32, c.c_int32, c.c_double]
    L.compams_create_in_workspace.restype = c.c_int
    L.compams_create_in_workspace.argtypes = [c.POINTER(H), c.c_void_p, c.c_size_t, c.c_int32, c.c_int32, c.c_int32,
                                              c.c_int64, c.POINTER(c.c_int64), c.c_int32, c.c_int32, c.c_double,
                                              c.c_float, c.c_float, c.c_float, c.c_float]
    L.compams_compress.restype = c.c_int
    L.compams_compress.argtypes = [H, c.c_void_p]
    L.compams_apply.restype = c.c_int
    L.compams_apply.argtypes = [H, c.c_void_p]
    L.compams_destroy.restype = c.c_int
    L.compams_destroy.argtypes = [H]
    L.compams_set_stream.restype = c.c_int
    L.compams_set_stream.argtypes = [H, c.c_void_p]
    L.compams_set_seed.restype = c.c_int
    L.compams_set_seed.argtypes = [H, c.c_uint64, c.c_uint64]
    L.compams_record_average.restype = c.c_int
    L.compams_record_average.argtypes = [H, c.c_int]
    L.compams_set_lr.restype = c.c_int
    L.compams_set_lr.argtypes = [H, c.c_float]
    L.compams_get_state.restype = c.c_int
    L.compams_get_state.argtypes = [H, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
    L.compams_set_state.restype = c.c_int
    L.compams_set_state.argtypes = [H, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
    L.compams_bits_transmitted.restype = c.c_int
    L.compams_bits_transmitted.argtypes = [H, c.POINTER(c.c_uint64)]
    L.compams_get_buffer.restype = c.c_int
    L.compams_get_buffer.argtypes = [H, c.c_int32, c.POINTER(c.c_void_p), c.POINTER(c.c_int64)]
    L.compams_check_status.restype = c.c_int
    L.compams_check_status.argtypes = [H, c.POINTER(c.c_uint32)]
    L.compams_set_profiling.restype = c.c_int
    L.compams_set_profiling.argtypes = [H, c.c_uint32]
    L.compams_get_kernel_time.restype = c.c_int
    L.compams_get_kernel_time.argtypes = [H, c.c_int32, c.POINTER(c.c_double), c.POINTER(c.c_int64)]
    L.compams_launch_count.restype = c.c_int64
    L.compams_launch_count.argtypes = [H]
    L.compams_blocksign_sweep_static.restype = c.c_int
    L.compams_blocksign_sweep_static.argtypes = [c.c_void_p] * 5 + [c.c_int32, c.c_int64, c.c_int32, c.c_void_p]
    L.compams_blocksign_sweep_static_limits.restype = c.c_int
    L.compams_blocksign_sweep_static_limits.argtypes = [c.POINTER(c.c_int64), c.POINTER(c.c_int64)]
    L.compams_error_string.restype = c.c_char_p
    L.compams_error_string.argtypes = [c.c_int]
    L.compams_kernel_name.restype = c.c_char_p
    L.compams_kernel_name.argtypes = [c.c_int32]
    L.compams_last_cuda_error.restype = c.c_char_p
    L.compams_last_cuda_error.argtypes = []
    _lib = L
    return L


def _check(rc: int, what: str) -> None:
    if rc != 0:
        L = load_library()
        msg = L.compams_error_string(rc).decode()
        cuda = L.compams_last_cuda_error().decode()
        raise CompAMSError("%s failed: %s (%d)%s" % (what, msg, rc, (" [" + cuda + "]") if cuda else ""))


def blocksign_sweep_static(grads: torch.Tensor, x_state: torch.Tensor, scales_prev: Optional[torch.Tensor],
                           scales_out: torch.Tensor, sign_bits: torch.Tensor, deferred: bool,
                           stream: Optional[torch.cuda.Stream] = None) -> None:
    """compams_blocksign_sweep_static: the Block-Sign sweep over one block per worker row, for callers
    that cannot allocate device memory. Every buffer is the caller's; nothing is allocated here either
    (the arguments are passed as raw pointers). See include/compams.h for sizes and limits."""
    L = load_library()
    n, d = grads.shape
    for t in (grads, x_state, scales_out, sign_bits) + ((scales_prev,) if scales_prev is not None else ()):
        if not (t.is_cuda and t.is_contiguous()):
            raise CompAMSError("blocksign_sweep_static takes contiguous CUDA tensors")
    if x_state.shape != grads.shape or scales_out.numel() != n or sign_bits.numel() != n * ((d + 31) // 32):
        raise CompAMSError("blocksign_sweep_static: buffer shapes do not match [n, d]")
    s = stream if stream is not None else torch.cuda.current_stream()
    rc = L.compams_blocksign_sweep_static(
        ctypes.c_void_p(grads.data_ptr()), ctypes.c_void_p(x_state.data_ptr()),
        ctypes.c_void_p(scales_prev.data_ptr() if scales_prev is not None else 0),
        ctypes.c_void_p(scales_out.data_ptr()), ctypes.c_void_p(sign_bits.data_ptr()), int(n), int(d),
        1 if deferred else 0, ctypes.c_void_p(s.cuda_stream))
    _check(rc, "compams_blocksign_sweep_static")


def blocksign_sweep_static_limits():
    """(max workers, max n * ceil(d / 8192)) accepted by blocksign_sweep_static."""
    a, b = ctypes.c_int64(), ctypes.c_int64()
    _check(load_library().compams_blocksign_sweep_static_limits(ctypes.byref(a), ctypes.byref(b)),
           "compams_blocksign_sweep_static_limits")
    return int(a.value), int(b.value)


def workspace_bytes(n: int, d: int, block_offsets: Sequence[int], compressor: int, k_ratio: float = 1.0,
                    n_total: Optional[int] = None) -> int:
    """Bytes of device memory a CompAMS of this shape needs when its state lives in caller memory
    (CompAMS(..., workspace=tensor)). Host arithmetic only: works without a GPU."""
    offs = np.ascontiguousarray(block_offsets, dtype=np.int64)
    out = ctypes.c_size_t(0)
    _check(load_library().compams_workspace_bytes(ctypes.byref(out), int(n), int(n if n_total is None else n_total), int(d),
                                                  offs.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), int(offs.size - 1),
                                                  int(compressor), float(k_ratio)), "compams_workspace_bytes")
    return int(out.value)


class _DeviceView:
    """Exposes a raw device pointer to torch through the CUDA array interface."""

    def __init__(self, ptr: int, count: int, dtype: torch.dtype, owner):
        self.__cuda_array_interface__ = {
            "shape": (count,), "typestr": _TYPESTR[dtype], "data": (ptr, False), "version": 2, "strides": None,
        }
        self._owner = owner


class CompAMS:
    """One COMP-AMS optimizer (Algorithm 2) on the current CUDA device.

    `step(grads, theta)` takes device tensors; `step_host(grads, theta)` takes host tensors and
    includes the transfers. `buffer(name)` returns a torch view of a library-owned device buffer.
    """

    def __init__(self, n: int, d: int, block_offsets: Sequence[int], compressor: int, k_ratio: float = 1.0,
                 lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                 stream: Optional[torch.cuda.Stream] = None, n_total: Optional[int] = None, first_worker: int = 0,
                 workspace: Optional[torch.Tensor] = None, record_average: bool = False):
        """`n` workers live in this optimizer. With `n_total` > n they are workers `first_worker` ...
        `first_worker + n - 1` of a job whose other workers live in other optimizers (other GPUs): use
        compress() / apply() with an exchange of the message buffers in between instead of step().
        `workspace`: a contiguous CUDA uint8 tensor of at least workspace_bytes(...) bytes, 256-byte aligned,
        that holds all of the optimizer's state (kept alive by this object); None: the library allocates.
        `record_average`: also store the averaged compressed gradient (buffer("gbar")); off, the update writes
        4 bytes per coordinate less."""
        self._L = load_library()
        self.n, self.d = int(n), int(d)
        self.n_total = self.n if n_total is None else int(n_total)
        self.first_worker = int(first_worker)
        offs = np.ascontiguousarray(block_offsets, dtype=np.int64)
        self.M = int(offs.size - 1)
        self.compressor = int(compressor)
        self._h = ctypes.c_void_p()
        self._workspace = workspace
        shape = (self.n, self.n_total, self.first_worker, self.d, offs.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                 self.M, self.compressor, float(k_ratio), float(lr), float(beta1), float(beta2), float(eps))
        if workspace is None:
            rc = self._L.compams_create_sharded(ctypes.byref(self._h), *shape)
        else:
            if not (workspace.is_cuda and workspace.dtype == torch.uint8 and workspace.is_contiguous()):
                raise CompAMSError("workspace must be a contiguous CUDA uint8 tensor")
            rc = self._L.compams_create_in_workspace(ctypes.byref(self._h), ctypes.c_void_p(workspace.data_ptr()),
                                                     int(workspace.numel()), *shape)
        if rc != 0:
            self._h = ctypes.c_void_p()
        _check(rc, "compams_create_sharded" if workspace is None else "compams_create_in_workspace")
        self.set_stream(stream if stream is not None else torch.cuda.current_stream())
        if record_average:
            self.record_average(True)

    # -- calls ---------------------------------------------------------------------------------
    def set_stream(self, stream: torch.cuda.Stream) -> None:
        _check(self._L.compams_set_stream(self._h, ctypes.c_void_p(stream.cuda_stream)), "compams_set_stream")

    def set_seed(self, seed: int, iterations_done: int = 0) -> None:
        """Random-k: the seed of the index sets and the number of iterations already done."""
        _check(self._L.compams_set_seed(self._h, int(seed), int(iterations_done)), "compams_set_seed")

    def record_average(self, on: bool = True) -> None:
        """Whether the following steps store the averaged compressed gradient, buffer("gbar")."""
        _check(self._L.compams_record_average(self._h, 1 if on else 0), "compams_record_average")

    def set_lr(self, lr: float) -> None:
        _check(self._L.compams_set_lr(self._h, float(lr)), "compams_set_lr")

    def get_state(self) -> dict:
        """The state Algorithm 2 carries between iterations, as new CUDA tensors: e [n, d]; m, v, vhat [d]."""
        dev = torch.device("cuda", torch.cuda.current_device())
        out = {"e": torch.empty(self.n, self.d, dtype=torch.float32, device=dev)}
        for name in ("m", "v", "vhat"):
            out[name] = torch.empty(self.d, dtype=torch.float32, device=dev)
        _check(self._L.compams_get_state(self._h, *(ctypes.c_void_p(out[k].data_ptr()) for k in ("e", "m", "v", "vhat"))),
               "compams_get_state")
        return out

    def set_state(self, state: dict) -> None:
        """Restore (part of) a state returned by get_state(); missing keys are left as they are."""
        ptrs = []
        for name, shape in (("e", (self.n, self.d)), ("m", (self.d,)), ("v", (self.d,)), ("vhat", (self.d,))):
            t = state.get(name)
            if t is None:
                ptrs.append(ctypes.c_void_p(0))
                continue
            if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == shape):
                raise CompAMSError("state[%r] must be a contiguous float32 CUDA tensor of shape %r" % (name, shape))
            ptrs.append(ctypes.c_void_p(t.data_ptr()))
        _check(self._L.compams_set_state(self._h, *ptrs), "compams_set_state")

    def bits_transmitted(self) -> dict:
        """Worker-to-server bits so far under the accounting of Section 5.2 (32 bits per float)."""
        out = (ctypes.c_uint64 * 3)()
        _check(self._L.compams_bits_transmitted(self._h, out), "compams_bits_transmitted")
        return {"full_precision": int(out[0]), "payload": int(out[1]), "topk_indices": int(out[2])}

    def step(self, grads: torch.Tensor, theta: torch.Tensor) -> None:
        if not (grads.is_cuda and theta.is_cuda):
            raise CompAMSError("step() takes CUDA tensors; use step_host() for host tensors")
        if grads.dtype not in (torch.float32, torch.bfloat16) or theta.dtype != torch.float32:
            raise CompAMSError("grads must be float32 or bfloat16, theta float32")
        if tuple(grads.shape) != (self.n, self.d) or not grads.is_contiguous():
            raise CompAMSError("grads must be a contiguous [n, d] tensor")
        if tuple(theta.shape) != (self.d,) or not theta.is_contiguous():
            raise CompAMSError("theta must be a contiguous [d] tensor")
        if grads.dtype == torch.bfloat16:
            _check(self._L.compams_step_bf16(self._h, ctypes.c_void_p(grads.data_ptr()),
                                             ctypes.c_void_p(theta.data_ptr())), "compams_step_bf16")
            return
        _check(self._L.compams_step(self._h, ctypes.c_void_p(grads.data_ptr()), ctypes.c_void_p(theta.data_ptr())),
               "compams_step")

    def compress(self, grads: torch.Tensor) -> None:
        """Worker side of one iteration (Algorithm 2, the workers' loop) for this optimizer's workers."""
        if not (grads.is_cuda and grads.dtype in (torch.float32, torch.bfloat16) and grads.is_contiguous()
                and tuple(grads.shape) == (self.n, self.d)):
            raise CompAMSError("grads must be a contiguous float32 or bfloat16 CUDA tensor of shape [n, d]")
        fn = self._L.compams_compress_bf16 if grads.dtype == torch.bfloat16 else self._L.compams_compress
        _check(fn(self._h, ctypes.c_void_p(grads.data_ptr())), "compams_compress")

    def apply(self, theta: torch.Tensor) -> None:
        """Server side (the server's part) over the messages of all n_total workers."""
        if not (theta.is_cuda and theta.dtype == torch.float32 and theta.is_contiguous()
                and tuple(theta.shape) == (self.d,)):
            raise CompAMSError("theta must be a contiguous float32 CUDA tensor of shape [d]")
        _check(self._L.compams_apply(self._h, ctypes.c_void_p(theta.data_ptr())), "compams_apply")

    def message_buffers(self):
        """The buffers an exchange between shards has to complete, as [n_total, width] views: every
        shard has filled rows first_worker ... first_worker + n - 1. Ask after compress()."""
        names = ("topk_idx", "topk_val") if self.compressor in (TOPK, RANDK) else ("sign_bits", "scales")
        return [self.buffer(name) for name in names]

    def step_host(self, grads: torch.Tensor, theta: torch.Tensor) -> None:
        if grads.is_cuda or theta.is_cuda:
            raise CompAMSError("step_host() takes host tensors")
        if grads.dtype != torch.float32 or theta.dtype != torch.float32:
            raise CompAMSError("grads and theta must be float32")
        if tuple(grads.shape) != (self.n, self.d) or not grads.is_contiguous():
            raise CompAMSError("grads must be a contiguous [n, d] tensor")
        if tuple(theta.shape) != (self.d,) or not theta.is_contiguous():
            raise CompAMSError("theta must be a contiguous [d] tensor")
        _check(self._L.compams_step_host(self._h, ctypes.c_void_p(grads.data_ptr()),
                                         ctypes.c_void_p(theta.data_ptr())), "compams_step_host")

    def buffer(self, name: str) -> torch.Tensor:
        """Torch view of a library-owned device buffer (valid until the next step / close)."""
        which = BUFFERS[name]
        ptr = ctypes.c_void_p()
        cnt = ctypes.c_int64()
        _check(self._L.compams_get_buffer(self._h, which, ctypes.byref(ptr), ctypes.byref(cnt)),
               "compams_get_buffer")
        dt = _BUFFER_DTYPES[name]
        if cnt.value == 0 or not ptr.value:
            if name == "E":  # every k_b = d_b: the error accumulators are identically zero and not stored
                return torch.zeros(self.n, self.d, dtype=dt, device="cuda")
            return torch.empty(0, dtype=dt, device="cuda")
        t = torch.as_tensor(_DeviceView(ptr.value, cnt.value, dt, self), device="cuda")
        if name == "E":
            return t.view(self.n, self.d)
        if name in ("topk_idx", "topk_val", "sign_bits"):
            return t.view(self.n_total, -1)
        if name == "scales":
            return t.view(self.n_total, self.M)
        return t

    def check_status(self) -> int:
        word = ctypes.c_uint32(0)
        rc = self._L.compams_check_status(self._h, ctypes.byref(word))
        _check(rc, "compams_check_status (status word 0x%x)" % word.value)
        return int(word.value)

    def set_profiling(self, kernels: Sequence[str]) -> None:
        mask = 0
        for k in kernels:
            mask |= 1 << KERNELS[k]
        _check(self._L.compams_set_profiling(self._h, mask), "compams_set_profiling")

    def kernel_time(self, kernel: str):
        """(total device milliseconds, launches) of one kernel since set_profiling()."""
        ms = ctypes.c_double(0.0)
        cnt = ctypes.c_int64(0)
        _check(self._L.compams_get_kernel_time(self._h, KERNELS[kernel], ctypes.byref(ms), ctypes.byref(cnt)),
               "compams_get_kernel_time")
        return ms.value, int(cnt.value)

    def launch_count(self) -> int:
        return int(self._L.compams_launch_count(self._h))

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            self._L.compams_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
