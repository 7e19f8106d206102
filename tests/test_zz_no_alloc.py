"""slimspec_head_topk_static: the entry point for callers that cannot allocate device memory.

Such callers -- a serving loop whose memory pool already owns the device, a plugin whose host
runtime forbids driver allocations -- have no context to hand over, so the call works out of a
fixed scratch array inside the library.  It must give what the context-based entry point gives,
also on a second call that finds the first call's leftovers in that array, and must refuse sizes
the array cannot hold.  Collected last on purpose: a failure here does not hide the other tests.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2605_10453_b200 import binding, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _static(g, k):
    M = g["h"].shape[0]
    ids = torch.full((M, k), -1, dtype=torch.int32, device=DEV)
    lp = torch.full((M, k), float("nan"), dtype=torch.float32, device=DEV)
    binding.slimspec_head_topk_static(g["h"], g["A"], g["B"], k, ids, lp)
    torch.cuda.synchronize()
    return ids.cpu().numpy(), lp.cpu().numpy()


def test_static_scratch_entry_point_matches_context_entry_point_twice():
    ctx = binding.Context(max_M=8, max_d=4096, max_V=128256, max_k=32)
    ctx.force_path(binding.PATH_STREAM)
    # two different problems in a row: the second call inherits the first one's scratch contents
    cases = [(3, 2048, 256, 128256, 10, 0), (1, 512, 128, 8 * 1501, 7, 1), (8, 1024, 192, 8 * 2500, 32, 2)]
    for M, d, r, V, k, seed in cases:
        x = synth.make_inputs(M, d, r, V, seed=seed)
        g = {n: t.to(DEV) for n, t in x.items()}
        want_ids, want_lp = ctx.slimspec_head_topk(g["h"], g["A"], g["B"], k)
        torch.cuda.synchronize()
        assert ctx.last_error() == binding.OK
        for _ in range(2):
            ids, lp = _static(g, k)
            # same kernels, same order of operations: the tolerance of the parity tests is ample
            assert np.array_equal(ids, want_ids.cpu().numpy())
            assert np.max(np.abs(lp - want_lp.cpu().numpy())) <= 2e-2
    ctx.close()


def test_static_scratch_entry_point_matches_the_oracle():
    """The same entry point against the CPU oracle (not only against the context-based call)."""
    import oracle
    from parity import check_topk
    M, d, r, V, k = 3, 512, 128, 8 * 1501, 7
    x = synth.make_inputs(M, d, r, V, seed=13)
    g = {n: t.to(DEV) for n, t in x.items()}
    b = {n: oracle.bf16_bits(t) for n, t in x.items()}
    ref = oracle.head_topk(b["h"], b["A"], b["B"], k)
    for _ in range(2):
        ids, lp = _static(g, k)
        st = check_topk(ref, ids, lp)
        assert st["max_lp_err"] <= 1e-3


def test_static_scratch_entry_point_allocates_nothing_after_its_first_call():
    """One warm-up call sets the entry point up (symbol address, kernels loaded); after it, calls of
    every row-count class leave the device's free memory unchanged."""
    d, r, V, k = 512, 128, 8 * 1501, 7
    xs = {M: {n: t.to(DEV) for n, t in synth.make_inputs(M, d, r, V, seed=M).items()} for M in (1, 2, 4, 8)}
    outs = {M: (torch.empty((M, k), dtype=torch.int32, device=DEV), torch.empty((M, k), dtype=torch.float32, device=DEV))
            for M in xs}
    binding.slimspec_head_topk_static(xs[1]["h"], xs[1]["A"], xs[1]["B"], k, *outs[1])      # the warm-up
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for M in (1, 2, 4, 8):
        binding.slimspec_head_topk_static(xs[M]["h"], xs[M]["A"], xs[M]["B"], k, *outs[M])
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    lib = binding.load()
    g = {n: t.to(DEV) for n, t in synth.make_inputs(2, 64, 64, 800, seed=1).items()}
    ids = torch.empty((2, 4), dtype=torch.int32, device=DEV)
    lp = torch.empty((2, 4), dtype=torch.float32, device=DEV)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    call = lambda M, d, r, V, k: lib.slimspec_head_topk_static(p(g["h"]), p(g["A"]), p(g["B"]), M, d, r, V, k,
                                                                p(ids), p(lp), None)
    assert call(binding.STATIC_MAX_M + 1, 64, 64, 800, 4) == binding.ERR_STATIC_LIMIT
    assert call(2, 64, binding.STATIC_MAX_R + 16, 800, 4) == binding.ERR_STATIC_LIMIT
    assert call(2, 64, 64, 800, binding.STATIC_MAX_K + 1) == binding.ERR_STATIC_LIMIT
    assert call(2, 64, 64, 804, 4) == binding.ERR_ALIGN          # V not a multiple of 8
    assert call(0, 64, 64, 800, 4) == binding.ERR_DIM
    assert lib.slimspec_head_topk_static(None, p(g["A"]), p(g["B"]), 2, 64, 64, 800, 4, p(ids), p(lp), None) == binding.ERR_NULL
    assert "fixed scratch" in binding.strerror(binding.ERR_STATIC_LIMIT)
    assert call(2, 64, 64, 800, 4) == binding.OK
    torch.cuda.synchronize()
