"""Build the CUDA library (sm_100a only) in-tree with nvcc.  No JIT cache, no torch extension."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libslimspec.so")
SOURCES = ["api.cu", "generic.cu", "stream.cu", "noalloc.cu", "tensor.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared",
]


def _newest_source_mtime() -> float:
    paths = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC)]
    paths.append(os.path.join(os.path.dirname(_PKG), "include", "slimspec.h"))
    return max(os.path.getmtime(p) for p in paths)


def is_stale() -> bool:
    return (not os.path.exists(LIB_PATH)) or os.path.getmtime(LIB_PATH) < _newest_source_mtime()


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libslimspec.so next to this file; returns its path."""
    if not force and not is_stale():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB_PATH + ".tmp%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp]
    cmd += [os.path.join(_CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
