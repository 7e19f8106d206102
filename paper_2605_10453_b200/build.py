"""Build the CUDA library (sm_100a only) in-tree with nvcc.  No JIT cache, no torch extension."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libslimspec.so")
SOURCES = ["api.cu", "generic.cu", "stream.cu", "stream_fma.cu", "noalloc.cu", "tensor.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared",
]


STAMP_PATH = os.path.join(_PKG, "libslimspec.srchash")


def _source_hash() -> str:
    """SHA-256 over the sources the library is built from (file times do not survive a copy)."""
    import hashlib
    h = hashlib.sha256()
    paths = sorted(os.path.join(_CSRC, f) for f in os.listdir(_CSRC))
    paths.append(os.path.join(os.path.dirname(_PKG), "include", "slimspec.h"))
    for p in paths:
        h.update(os.path.basename(p).encode())
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def is_stale() -> bool:
    if not (os.path.exists(LIB_PATH) and os.path.exists(STAMP_PATH)):
        return True
    with open(STAMP_PATH) as f:
        return f.read().strip() != _source_hash()


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libslimspec.so next to this file; returns its path."""
    if not force and not is_stale():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB_PATH + ".tmp%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp]
    cmd += [os.path.join(_CSRC, s) for s in SOURCES]
    digest = _source_hash()
    subprocess.check_call(cmd)
    os.replace(tmp, LIB_PATH)
    with open(STAMP_PATH + ".tmp%d" % os.getpid(), "w") as f:
        f.write(digest + "\n")
    os.replace(STAMP_PATH + ".tmp%d" % os.getpid(), STAMP_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
