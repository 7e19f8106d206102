"""B200-native SlimSpec draft LM-head: low-rank head with fused log-softmax / top-k.

`binding` mirrors the C ABI of include/slimspec.h; `synth` draws the seeded workloads;
`build` compiles the CUDA sources in-tree for sm_100a.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]
