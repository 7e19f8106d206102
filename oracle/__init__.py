"""CPU fp64 oracle for the SlimSpec draft LM-head forward -- TEST INFRASTRUCTURE ONLY.

Thin ctypes binding over ``slimspec_oracle.c`` (plain C, fp64, optional OpenMP over rows).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library never does, and the two share no code.

All weight / activation arguments are numpy ``uint16`` arrays holding bf16 bit patterns
(``bf16_bits`` converts a torch bf16 tensor without changing a bit).  Conventions follow
Section 4.1 of the paper transposed to row vectors: ``h`` is M x d, ``A`` = W_down^T is
d x r, ``B`` = W_up^T is r x V, ``W`` = W_full^T is d x V.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "slimspec_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _bind(path):
    """Load one build of the oracle and declare its signatures."""
    lib = ctypes.CDLL(path)
    u16 = ctypes.POINTER(ctypes.c_uint16)
    f64 = ctypes.POINTER(ctypes.c_double)
    i32 = ctypes.POINTER(ctypes.c_int32)
    ci = ctypes.c_int
    lib.oracle_threads.restype = ci
    lib.oracle_set_threads.argtypes = [ci]
    lib.oracle_downproj.argtypes = [u16, u16, ci, ci, ci, f64]
    lib.oracle_upproj.argtypes = [f64, u16, ci, ci, ci, f64]
    lib.oracle_slimspec_logits.argtypes = [u16, u16, u16, ci, ci, ci, ci, f64]
    lib.oracle_slimspec_logits.restype = ci
    lib.oracle_fullhead_logits.argtypes = [u16, u16, ci, ci, ci, f64]
    lib.oracle_log_softmax.argtypes = [f64, ci, ci, f64, f64]
    lib.oracle_topk.argtypes = [f64, ci, ci, ci, i32, f64, f64]
    lib.oracle_topk.restype = ci
    return lib


def _load():
    global _lib
    if _lib is None:
        _lib = _bind(build())
    return _lib


def _u16(a, shape):
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16 or a.shape != tuple(shape):
        raise ValueError("expected uint16 bf16 bits of shape %s, got %s %s" % (shape, a.dtype, a.shape))
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))


def _f64p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def bf16_bits(t) -> np.ndarray:
    """Bit pattern of a torch bf16 tensor (CPU or CUDA) as a numpy uint16 array."""
    import torch

    if t.dtype != torch.bfloat16:
        raise ValueError("bf16_bits wants a bfloat16 tensor")
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def threads() -> int:
    return int(_load().oracle_threads())


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


def downproj(h, A) -> np.ndarray:
    """z = h A in fp64 (Section 4.1, W_down h).  Returns M x r."""
    M, d = h.shape
    r = A.shape[1]
    h, hp = _u16(h, (M, d))
    A, Ap = _u16(A, (d, r))
    z = np.empty((M, r), dtype=np.float64)
    _load().oracle_downproj(hp, Ap, M, d, r, _f64p(z))
    return z


def slimspec_logits(h, A, B) -> np.ndarray:
    """logits = (h A) B in fp64 (Section 4.1, W_up W_down h).  Returns M x V."""
    M, d = h.shape
    r, V = B.shape
    h, hp = _u16(h, (M, d))
    A, Ap = _u16(A, (d, r))
    B, Bp = _u16(B, (r, V))
    out = np.empty((M, V), dtype=np.float64)
    rc = _load().oracle_slimspec_logits(hp, Ap, Bp, M, d, r, V, _f64p(out))
    if rc != 0:
        raise MemoryError("oracle_slimspec_logits failed (%d)" % rc)
    return out


def fullhead_logits(h, W) -> np.ndarray:
    """logits = h W in fp64 (Section 4.1, W_full h).  Returns M x V."""
    M, d = h.shape
    V = W.shape[1]
    h, hp = _u16(h, (M, d))
    W, Wp = _u16(W, (d, V))
    out = np.empty((M, V), dtype=np.float64)
    _load().oracle_fullhead_logits(hp, Wp, M, d, V, _f64p(out))
    return out


def log_softmax(logits):
    """Row-wise stable log-softmax in fp64.  Returns (logprob M x V, lse M)."""
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    M, V = logits.shape
    lp = np.empty_like(logits)
    lse = np.empty(M, dtype=np.float64)
    _load().oracle_log_softmax(_f64p(logits), M, V, _f64p(lp), _f64p(lse))
    return lp, lse


def topk(vals, k: int):
    """Top-k by full sort, (value desc, id asc).  Returns (ids M x k int32, vals M x k, next M)."""
    vals = np.ascontiguousarray(vals, dtype=np.float64)
    M, V = vals.shape
    ids = np.empty((M, k), dtype=np.int32)
    top = np.empty((M, k), dtype=np.float64)
    nxt = np.empty(M, dtype=np.float64)
    rc = _load().oracle_topk(_f64p(vals), M, V, int(k),
                             ids.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), _f64p(top), _f64p(nxt))
    if rc != 0:
        raise ValueError("oracle_topk failed (%d)" % rc)
    return ids, top, nxt


def head_topk(h, A, B, k: int):
    """The whole low-rank path.  Returns dict(ids, logprobs, logits, logprob_full, lse, next_logit)."""
    return _finish(slimspec_logits(h, A, B), k)


def fullhead_topk(h, W, k: int):
    """The whole standard-head path; same result layout as head_topk."""
    return _finish(fullhead_logits(h, W), k)


def _finish(logits, k):
    lp, lse = log_softmax(logits)
    ids, top, nxt = topk(logits, k)
    return {
        "ids": ids,
        "logprobs": top - lse[:, None],
        "logits": logits,
        "logprob_full": lp,
        "lse": lse,
        "top_logits": top,
        "next_logit": nxt,
    }
