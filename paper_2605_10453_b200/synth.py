"""Seeded synthetic inputs for the draft LM-head workloads.

This module only draws numbers; it contains none of the head's arithmetic, so both the
CUDA tests and the CPU oracle's tests may use it.  Every tensor has its own CPU generator
(seed * 1000003 + tag), so leaving one tensor out does not change the others:

    h ~ N(0, 1)        M x d     tag 1
    A ~ N(0, 1/d)      d x r     tag 2      (W_down^T of Section 4.1)
    B ~ N(0, 1/r)      r x V     tag 3      (W_up^T), optionally times ``logit_scale``
    W ~ N(0, 1/d)      d x V     tag 4      (W_full^T, the standard head)

Each is drawn in fp32 in row blocks of ``_ROWS_PER_DRAW`` rows (the block order is part of
the recipe), scaled, and rounded once to bf16.  ``logit_scale`` must be a power of two so
that the scaling is exact in bf16.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

_ROWS_PER_DRAW = 256


@dataclass(frozen=True)
class HeadConfig:
    name: str
    d: int
    r: int
    V: int
    k: int
    Ms: tuple
    logit_scale: float = 1.0
    seed: int = 0


# The workloads of the benchmark spec: a tiny case, an 8B-class head, a larger-vocabulary
# head with sharpened logits, and a throughput batch (64 sequences x 8 draft-tree nodes).
CONFIGS = {
    "c0": HeadConfig("c0", d=2048, r=256, V=128256, k=10, Ms=(1,)),
    "c1": HeadConfig("c1", d=4096, r=512, V=128256, k=10, Ms=(1, 8)),
    "c2": HeadConfig("c2", d=5120, r=640, V=152064, k=8, Ms=(1, 16), logit_scale=4.0),
    "c3": HeadConfig("c3", d=4096, r=512, V=128256, k=10, Ms=(512,)),
}
SWEEP_D = 8192
SWEEP_V = 128256
SWEEP_RANKS = (512, 1024, 2048)
SWEEP_MS = (1, 4, 16, 64, 256, 1024)


def sweep_config(r: int) -> HeadConfig:
    return HeadConfig("c4_r%d" % r, d=SWEEP_D, r=r, V=SWEEP_V, k=10, Ms=SWEEP_MS)


def _draw(rows: int, cols: int, std: float, seed: int, tag: int) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed * 1000003 + tag)
    out = torch.empty((rows, cols), dtype=torch.bfloat16)
    for r0 in range(0, rows, _ROWS_PER_DRAW):
        n = min(_ROWS_PER_DRAW, rows - r0)
        blk = torch.randn((n, cols), generator=g, dtype=torch.float32)
        out[r0:r0 + n] = (blk * std).to(torch.bfloat16)
    return out


def make_h(M: int, d: int, seed: int = 0) -> torch.Tensor:
    return _draw(M, d, 1.0, seed, 1)


def make_A(d: int, r: int, seed: int = 0) -> torch.Tensor:
    return _draw(d, r, 1.0 / math.sqrt(d), seed, 2)


def make_B(r: int, V: int, seed: int = 0, logit_scale: float = 1.0) -> torch.Tensor:
    if logit_scale <= 0 or math.frexp(logit_scale)[0] != 0.5:
        raise ValueError("logit_scale must be a positive power of two")
    return _draw(r, V, logit_scale / math.sqrt(r), seed, 3)


def make_W(d: int, V: int, seed: int = 0) -> torch.Tensor:
    return _draw(d, V, 1.0 / math.sqrt(d), seed, 4)


def make_inputs(M: int, d: int, r: int, V: int, seed: int = 0, logit_scale: float = 1.0,
                full: bool = False):
    """dict(h, A, B[, W]) of CPU bf16 tensors."""
    out = {
        "h": make_h(M, d, seed),
        "A": make_A(d, r, seed),
        "B": make_B(r, V, seed, logit_scale),
    }
    if full:
        out["W"] = make_W(d, V, seed)
    return out
