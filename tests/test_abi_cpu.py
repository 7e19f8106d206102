"""CPU-side checks of the boundary: the library builds, loads and exports what the header declares."""
import ctypes
import os
import re

import pytest

from paper_2605_10453_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "slimspec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b([a-z_0-9]+)\s*\(", text)
    return sorted({n for n in names if n.startswith(("slimspec_", "fullhead_"))})


def test_header_and_binding_agree():
    assert declared_functions() == sorted(binding.EXPORTS)


def test_library_exports_every_declared_symbol(lib):
    raw = ctypes.CDLL(binding.lib_path())
    for name in declared_functions():
        assert hasattr(raw, name), name


def test_strerror_without_gpu(lib):
    assert binding.strerror(binding.OK) == "ok"
    seen = {binding.strerror(c) for c in range(-6, 1)}
    assert len(seen) == 7
    assert "unknown" in binding.strerror(-99)


def test_create_rejects_bad_arguments_before_touching_cuda(lib):
    h = ctypes.c_void_p()
    assert lib.slimspec_create(None, 1, 1, 1, 1) == binding.ERR_NULL
    assert lib.slimspec_create(ctypes.byref(h), 0, 8, 8, 1) == binding.ERR_DIM
    assert lib.slimspec_create(ctypes.byref(h), 1, 8, 8, binding.MAX_K + 1) == binding.ERR_DIM
    assert h.value is None


def test_null_context_is_an_error_not_a_crash(lib):
    assert lib.slimspec_force_path(None, 0) == binding.ERR_NULL
    assert lib.slimspec_last_error(None) == binding.ERR_NULL
    assert lib.slimspec_head_topk(None, None, None, None, 1, 1, 1, 1, 1, None, None, None) == binding.ERR_NULL
    lib.slimspec_destroy(None)
