"""ctypes binding of libslimspec.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every step of the head runs in the library's
CUDA kernels.  If the library is missing this module raises -- there is no fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

OK = 0
ERR_NULL, ERR_DIM, ERR_ALIGN, ERR_CUDA, ERR_TIMEOUT, ERR_NOMEM = -1, -2, -3, -4, -5, -6
ERR_STATIC_LIMIT = -7
STATIC_MAX_M, STATIC_MAX_R, STATIC_MAX_K = 8, 8192, 32
PATH_AUTO, PATH_GENERIC, PATH_STREAM, PATH_TENSOR = 0, 1, 2, 3
MAX_K = 64

EXPORTS = [
    "slimspec_create", "slimspec_destroy", "slimspec_force_path", "slimspec_last_path",
    "slimspec_head_topk", "slimspec_head_topk_host", "slimspec_head_logits", "fullhead_topk",
    "slimspec_last_error", "slimspec_launch_count", "slimspec_strerror",
    "slimspec_kernel_timing", "slimspec_kernel_timing_read", "slimspec_head_topk_static",
]

_lib = None


class SlimSpecError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__("%s: %s (%d)" % (what, strerror(status), status))


def lib_path() -> str:
    return _build.LIB_PATH


def load():
    """Load the shared library (must have been built: see build.py); declares signatures."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError("libslimspec.so is not built; run `python -m paper_2605_10453_b200.build`")
    lib = ctypes.CDLL(path)
    vp, ci = ctypes.c_void_p, ctypes.c_int
    lib.slimspec_create.argtypes = [ctypes.POINTER(vp), ci, ci, ci, ci]
    lib.slimspec_create.restype = ci
    lib.slimspec_destroy.argtypes = [vp]
    lib.slimspec_destroy.restype = None
    lib.slimspec_force_path.argtypes = [vp, ci]
    lib.slimspec_force_path.restype = ci
    lib.slimspec_last_path.argtypes = [vp]
    lib.slimspec_last_path.restype = ci
    lib.slimspec_head_topk.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, vp, vp, vp]
    lib.slimspec_head_topk.restype = ci
    lib.slimspec_head_topk_host.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, vp, vp, vp]
    lib.slimspec_head_topk_host.restype = ci
    lib.slimspec_head_logits.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, vp, vp]
    lib.slimspec_head_logits.restype = ci
    lib.fullhead_topk.argtypes = [vp, vp, vp, ci, ci, ci, ci, vp, vp, vp]
    lib.fullhead_topk.restype = ci
    lib.slimspec_last_error.argtypes = [vp]
    lib.slimspec_last_error.restype = ci
    lib.slimspec_launch_count.argtypes = [vp]
    lib.slimspec_launch_count.restype = ctypes.c_longlong
    lib.slimspec_kernel_timing.argtypes = [vp, ci]
    lib.slimspec_kernel_timing.restype = ci
    lib.slimspec_kernel_timing_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double),
                                                ctypes.POINTER(ctypes.c_longlong)]
    lib.slimspec_kernel_timing_read.restype = ci
    lib.slimspec_head_topk_static.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, vp, vp, vp]
    lib.slimspec_head_topk_static.restype = ci
    lib.slimspec_strerror.argtypes = [ci]
    lib.slimspec_strerror.restype = ctypes.c_char_p
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load().slimspec_strerror(int(status)).decode()


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check_dev(t, dtype, shape, name):
    if not t.is_cuda or t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA %s tensor of shape %s" % (name, dtype, tuple(shape)))


class Context:
    """Owns one slimspec_ctx (scratch for calls up to the given sizes) on the current device."""

    def __init__(self, max_M: int, max_d: int, max_V: int, max_k: int = 32):
        self._h = ctypes.c_void_p()
        rc = load().slimspec_create(ctypes.byref(self._h), max_M, max_d, max_V, max_k)
        if rc != OK:
            raise SlimSpecError(rc, "slimspec_create")

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            load().slimspec_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def force_path(self, path: int):
        rc = load().slimspec_force_path(self._h, path)
        if rc != OK:
            raise SlimSpecError(rc, "slimspec_force_path")

    def last_path(self) -> int:
        return load().slimspec_last_path(self._h)

    def last_error(self) -> int:
        return load().slimspec_last_error(self._h)

    def launch_count(self) -> int:
        return int(load().slimspec_launch_count(self._h))

    def kernel_timing(self, enable: bool):
        rc = load().slimspec_kernel_timing(self._h, 1 if enable else 0)
        if rc != OK:
            raise SlimSpecError(rc, "slimspec_kernel_timing")

    def kernel_timing_read(self):
        """(total milliseconds, launches) of the timed dominant kernel since timing was enabled."""
        ms, n = ctypes.c_double(), ctypes.c_longlong()
        rc = load().slimspec_kernel_timing_read(self._h, ctypes.byref(ms), ctypes.byref(n))
        if rc != OK:
            raise SlimSpecError(rc, "slimspec_kernel_timing_read")
        return ms.value, int(n.value)

    # ---- the calls of the C ABI; outputs may be passed in to avoid allocation -----------
    def slimspec_head_topk(self, h, A, B, k, out_ids=None, out_logprobs=None, stream=None):
        M, d = h.shape
        r, V = B.shape
        _check_dev(h, torch.bfloat16, (M, d), "h")
        _check_dev(A, torch.bfloat16, (d, r), "A")
        _check_dev(B, torch.bfloat16, (r, V), "B")
        if out_ids is None:
            out_ids = torch.empty((M, k), dtype=torch.int32, device=h.device)
        if out_logprobs is None:
            out_logprobs = torch.empty((M, k), dtype=torch.float32, device=h.device)
        _check_dev(out_ids, torch.int32, (M, k), "out_ids")
        _check_dev(out_logprobs, torch.float32, (M, k), "out_logprobs")
        rc = load().slimspec_head_topk(self._h, _ptr(h), _ptr(A), _ptr(B), M, d, r, V, k,
                                       _ptr(out_ids), _ptr(out_logprobs), _stream(stream))
        if rc != OK:
            raise SlimSpecError(rc, "slimspec_head_topk")
        return out_ids, out_logprobs

    def slimspec_head_topk_host(self, h_host, A, B, k, out_ids_host=None, out_logprobs_host=None, stream=None):
        M, d = h_host.shape
        r, V = B.shape
        if h_host.is_cuda or h_host.dtype != torch.bfloat16 or not h_host.is_contiguous():
            raise ValueError("h_host must be a contiguous CPU bf16 tensor")
        _check_dev(A, torch.bfloat16, (d, r), "A")
        _check_dev(B, torch.bfloat16, (r, V), "B")
        if out_ids_host is None:
            out_ids_host = torch.empty((M, k), dtype=torch.int32).pin_memory()
        if out_logprobs_host is None:
            out_logprobs_host = torch.empty((M, k), dtype=torch.float32).pin_memory()
        rc = load().slimspec_head_topk_host(self._h, _ptr(h_host), _ptr(A), _ptr(B), M, d, r, V, k,
                                            _ptr(out_ids_host), _ptr(out_logprobs_host), _stream(stream))
        if rc != OK:
            raise SlimSpecError(rc, "slimspec_head_topk_host")
        return out_ids_host, out_logprobs_host

    def slimspec_head_logits(self, h, A, B, out_logits=None, stream=None):
        M, d = h.shape
        r, V = B.shape
        _check_dev(h, torch.bfloat16, (M, d), "h")
        _check_dev(A, torch.bfloat16, (d, r), "A")
        _check_dev(B, torch.bfloat16, (r, V), "B")
        if out_logits is None:
            out_logits = torch.empty((M, V), dtype=torch.float32, device=h.device)
        _check_dev(out_logits, torch.float32, (M, V), "out_logits")
        rc = load().slimspec_head_logits(self._h, _ptr(h), _ptr(A), _ptr(B), M, d, r, V,
                                         _ptr(out_logits), _stream(stream))
        if rc != OK:
            raise SlimSpecError(rc, "slimspec_head_logits")
        return out_logits

    def fullhead_topk(self, h, W, k, out_ids=None, out_logprobs=None, stream=None):
        M, d = h.shape
        V = W.shape[1]
        _check_dev(h, torch.bfloat16, (M, d), "h")
        _check_dev(W, torch.bfloat16, (d, V), "W")
        if out_ids is None:
            out_ids = torch.empty((M, k), dtype=torch.int32, device=h.device)
        if out_logprobs is None:
            out_logprobs = torch.empty((M, k), dtype=torch.float32, device=h.device)
        rc = load().fullhead_topk(self._h, _ptr(h), _ptr(W), M, d, V, k,
                                  _ptr(out_ids), _ptr(out_logprobs), _stream(stream))
        if rc != OK:
            raise SlimSpecError(rc, "fullhead_topk")
        return out_ids, out_logprobs


def slimspec_head_topk_static(h, A, B, k, out_ids, out_logprobs, stream=None):
    """slimspec_head_topk_static of the C ABI: no context, no allocation (here neither: the
    caller passes the output tensors).  For callers that must not allocate device memory --
    a serving loop whose pool owns the device, a plugin under a runtime that forbids driver
    allocations.  M <= 8, r <= 8192, k <= 32; calls that overlap on the GPU race on the
    library's one static scratch array."""
    M, d = h.shape
    r, V = B.shape
    _check_dev(h, torch.bfloat16, (M, d), "h")
    _check_dev(A, torch.bfloat16, (d, r), "A")
    _check_dev(B, torch.bfloat16, (r, V), "B")
    _check_dev(out_ids, torch.int32, (M, k), "out_ids")
    _check_dev(out_logprobs, torch.float32, (M, k), "out_logprobs")
    rc = load().slimspec_head_topk_static(_ptr(h), _ptr(A), _ptr(B), M, d, r, V, k,
                                          _ptr(out_ids), _ptr(out_logprobs), _stream(stream))
    if rc != OK:
        raise SlimSpecError(rc, "slimspec_head_topk_static")
    return out_ids, out_logprobs
