"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU oracle, same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_10453_b200 import binding, synth
from parity import LOGPROB_TOL, check_topk

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def dev(x):
    return {k: v.to(DEV) for k, v in x.items()}


def obits(x):
    return {k: oracle.bf16_bits(v) for k, v in x.items()}


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(max_M=512, max_d=8192, max_V=160000, max_k=64)
    yield c
    c.close()


def run_topk(ctx, x, k, path):
    ctx.force_path(path)
    g = dev(x)
    ids, lp = ctx.slimspec_head_topk(g["h"], g["A"], g["B"], k)
    torch.cuda.synchronize()
    assert ctx.last_error() == binding.OK
    assert ctx.last_path() == path
    return ids.cpu().numpy(), lp.cpu().numpy()


# ---------------------------------------------------------------- tiny and ragged shapes

GENERIC_SHAPES = [
    # M, d, r, V, k
    (1, 8, 2, 37, 5),
    (3, 8, 2, 37, 37),
    (5, 33, 7, 1001, 10),
    (2, 64, 16, 4099, 64),
    (17, 128, 24, 2500, 8),
]


@pytest.mark.parametrize("M,d,r,V,k", GENERIC_SHAPES)
def test_generic_path_any_shape(ctx, M, d, r, V, k):
    x = synth.make_inputs(M, d, r, V, seed=11)
    ids, lp = run_topk(ctx, x, k, binding.PATH_GENERIC)
    b = obits(x)
    st = check_topk(oracle.head_topk(b["h"], b["A"], b["B"], k), ids, lp)
    assert st["max_lp_err"] < 1e-3


STREAM_SHAPES = [
    # M, d, r, V, k  -- V/8 units vs 148 slabs: fewer units than slabs, ragged split, several passes
    (1, 64, 64, 8 * 100, 10),
    (1, 256, 64, 8 * 149, 10),
    (2, 512, 128, 8 * (148 * 3 + 5), 7),
    (3, 1000, 192, 8 * 1999, 10),
    (4, 2048, 256, 8 * 4001, 32),
    (5, 96, 64, 8 * 777, 1),
    (8, 1024, 128, 8 * 2500, 10),
    (7, 160, 320, 8 * 148 * 130, 5),      # 130 units per slab: two column passes
    (11, 512, 64, 8 * 1501, 10),          # two row tiles (8 + 3)
    (3, 8192, 512, 8 * 1501, 10),         # a large A: three and four rows take the one-launch kernel
    (4, 4096, 1024, 8 * 777, 5),
]


@pytest.mark.parametrize("M,d,r,V,k", STREAM_SHAPES)
def test_stream_path_matches_oracle(ctx, M, d, r, V, k):
    x = synth.make_inputs(M, d, r, V, seed=5)
    ids, lp = run_topk(ctx, x, k, binding.PATH_STREAM)
    b = obits(x)
    st = check_topk(oracle.head_topk(b["h"], b["A"], b["B"], k), ids, lp)
    assert st["max_lp_err"] < 1e-3
    # a second run must reproduce the first bit for bit (deterministic merge order)
    ids2, lp2 = run_topk(ctx, x, k, binding.PATH_STREAM)
    assert np.array_equal(ids, ids2) and np.array_equal(lp.view(np.uint32), lp2.view(np.uint32))
    # and the generic kernels, a second GPU implementation, agree too
    ids3, lp3 = run_topk(ctx, x, k, binding.PATH_GENERIC)
    assert np.max(np.abs(lp - lp3)) < 1e-3


def test_interleaved_shapes_share_the_scratch(ctx):
    """One context, calls of changing shape and row count back to back without a synchronisation in
    between: the one-launch kernel of one and two rows hands its code over through words in the
    context's scratch that carry the number of the call, and every streaming kernel counts its CTAs
    in on a counter that only counts up; neither may take a previous call's leftovers for its own."""
    cases = [(1, 256, 64, 8 * 149, 10), (2, 512, 128, 8 * 1337, 7), (5, 96, 64, 8 * 777, 3), (1, 64, 64, 8 * 100, 10),
             (16, 512, 64, 8 * 1501, 10), (2, 64, 64, 8 * 100, 5), (1, 512, 128, 8 * 1337, 7), (9, 256, 64, 8 * 149, 4)]
    ctx.force_path(binding.PATH_STREAM)
    inputs = [synth.make_inputs(M, d, r, V, seed=40 + i) for i, (M, d, r, V, k) in enumerate(cases)]
    gpu = [dev(x) for x in inputs]
    outs = []
    for rep in range(3):
        outs = []
        for (M, d, r, V, k), g in zip(cases, gpu):
            outs.append(ctx.slimspec_head_topk(g["h"], g["A"], g["B"], k))
    torch.cuda.synchronize()
    assert ctx.last_error() == binding.OK
    for (M, d, r, V, k), x, (ids, lp) in zip(cases, inputs, outs):
        b = obits(x)
        st = check_topk(oracle.head_topk(b["h"], b["A"], b["B"], k), ids.cpu().numpy(), lp.cpu().numpy())
        assert st["max_lp_err"] < 1e-3, (M, d, r, V, k)
    # the full-rank head of one and two rows goes through the same kernel (its code is h itself)
    for M in (1, 2):
        h = synth.make_h(M, 256, 9)
        W = synth.make_W(256, 8 * 901, 9)
        ids, lp = ctx.fullhead_topk(h.to(DEV), W.to(DEV), 6)
        torch.cuda.synchronize()
        st = check_topk(oracle.fullhead_topk(oracle.bf16_bits(h), oracle.bf16_bits(W), 6), ids.cpu().numpy(), lp.cpu().numpy())
        assert st["max_lp_err"] < 1e-3
    ctx.force_path(binding.PATH_AUTO)


def test_random_shapes_in_batches_against_oracle(ctx):
    """Seeded random shapes (rows 1..16, every streaming kernel and its variants by row count), enqueued six
    at a time without a synchronisation in between, twice over; every result against the oracle."""
    import random
    rng = random.Random(20260510)
    ctx.force_path(binding.PATH_AUTO)
    batch = []
    for it in range(24):
        M = rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 12, 15, 16])
        d = rng.choice([64, 128, 256, 520, 1024, 2048, 4096])
        r = rng.choice([16, 32, 64, 128, 256, 512])
        V = 8 * rng.randint(20, 2000)
        k = rng.randint(1, min(32, V))
        x = synth.make_inputs(M, d, r, V, seed=100 + it)
        batch.append((M, d, r, V, k, x, dev(x)))
        if len(batch) < 6:
            continue
        for rep in range(2):
            outs = [ctx.slimspec_head_topk(g["h"], g["A"], g["B"], k_) for (_, _, _, _, k_, _, g) in batch]
        torch.cuda.synchronize()
        assert ctx.last_error() == binding.OK
        for (M_, d_, r_, V_, k_, x_, _), (ids, lp) in zip(batch, outs):
            b = obits(x_)
            st = check_topk(oracle.head_topk(b["h"], b["A"], b["B"], k_), ids.cpu().numpy(), lp.cpu().numpy())
            assert st["max_lp_err"] < 1e-3, (M_, d_, r_, V_, k_)
        batch = []


TENSOR_SHAPES = [
    # M, d, r, V, k -- one and several row blocks, ragged last column tile, V below one tile
    (1, 64, 64, 64, 3),
    (9, 128, 64, 2048, 10),
    (40, 256, 128, 8 * 1501, 5),
    (128, 192, 64, 8 * 333, 32),
    (130, 512, 128, 8 * 2600, 10),
    (300, 256, 64, 20000, 1),
]


@pytest.mark.parametrize("M,d,r,V,k", TENSOR_SHAPES)
def test_tensor_path_matches_oracle(ctx, M, d, r, V, k):
    x = synth.make_inputs(M, d, r, V, seed=3)
    ids, lp = run_topk(ctx, x, k, binding.PATH_TENSOR)
    b = obits(x)
    st = check_topk(oracle.head_topk(b["h"], b["A"], b["B"], k), ids, lp)
    assert st["max_lp_err"] <= LOGPROB_TOL
    ids2, lp2 = run_topk(ctx, x, k, binding.PATH_TENSOR)
    assert np.array_equal(ids, ids2) and np.array_equal(lp.view(np.uint32), lp2.view(np.uint32))
    # raw logits through the same kernels, canaries around the output
    g = dev(x)
    ctx.force_path(binding.PATH_TENSOR)
    buf = torch.full((M * V + 512,), 12345.0, dtype=torch.float32, device=DEV)
    out = buf[256:256 + M * V].view(M, V)
    ctx.slimspec_head_logits(g["h"], g["A"], g["B"], out_logits=out)
    torch.cuda.synchronize()
    assert ctx.last_error() == binding.OK and ctx.last_path() == binding.PATH_TENSOR
    assert torch.all(buf[:256] == 12345.0) and torch.all(buf[256 + M * V:] == 12345.0)
    ref = oracle.slimspec_logits(b["h"], b["A"], b["B"])
    assert np.max(np.abs(out.cpu().numpy().astype(np.float64) - ref)) <= 2e-2


def test_tensor_path_fullhead_and_planted_tie(ctx):
    M, d, V, k = 70, 256, 8 * 1200, 6
    h = synth.make_h(M, d, 5)
    W = synth.make_W(d, V, 5)
    ref = oracle.fullhead_topk(oracle.bf16_bits(h), oracle.bf16_bits(W), k)
    best = int(ref["ids"][0, 0])
    twin = (best + 4099) % V
    W[:, twin] = W[:, best]
    ref = oracle.fullhead_topk(oracle.bf16_bits(h), oracle.bf16_bits(W), k)
    ctx.force_path(binding.PATH_AUTO)
    ids, lp = ctx.fullhead_topk(h.to(DEV), W.to(DEV), k)
    torch.cuda.synchronize()
    assert ctx.last_error() == binding.OK and ctx.last_path() == binding.PATH_TENSOR
    ids, lp = ids.cpu().numpy(), lp.cpu().numpy()
    st = check_topk(ref, ids, lp)
    assert st["max_lp_err"] <= 1e-3        # h is exact in bf16: only fp32 accumulation differs
    assert ids[0, :2].tolist() == sorted([best, twin]) and lp[0, 0] == lp[0, 1]


@pytest.mark.parametrize("M,k", [(6, 10), (140, 10), (70, 32)])
def test_tensor_path_ascending_logits_fill_the_candidate_lists(ctx, M, k):
    """Logits that grow with the column index: the bound taken from the first tiles prunes nothing,
    nearly every later column is a candidate, so the per-row lists overflow and are compacted over
    and over; runs of equal bf16 weights give ties that must resolve to the lower id."""
    d, V = 64, 8 * 1400
    g = torch.Generator().manual_seed(19)
    h = (torch.rand((M, d), generator=g) * 0.5 + 0.25).to(torch.bfloat16)
    s = torch.rand((d, 1), generator=g) * 0.2 + 0.05
    W = (s * ((torch.arange(V, dtype=torch.float32) + 1.0) / V).view(1, V)).to(torch.bfloat16)
    ref = oracle.fullhead_topk(oracle.bf16_bits(h), oracle.bf16_bits(W), k)
    assert np.all(np.diff(ref["logits"], axis=1) >= 0)            # ascending, with ties
    ctx.force_path(binding.PATH_TENSOR)
    ids, lp = ctx.fullhead_topk(h.to(DEV), W.to(DEV), k)
    torch.cuda.synchronize()
    assert ctx.last_error() == binding.OK and ctx.last_path() == binding.PATH_TENSOR
    ids, lp = ids.cpu().numpy(), lp.cpu().numpy()
    st = check_topk(ref, ids, lp)
    assert st["max_lp_err"] <= 1e-3
    # among equal logits the lower id comes first
    for m in range(M):
        for j in range(k - 1):
            if lp[m, j] == lp[m, j + 1]:
                assert ids[m, j] < ids[m, j + 1]
    ctx.force_path(binding.PATH_AUTO)


def test_stream_path_refuses_what_it_cannot_take(ctx):
    x = dev(synth.make_inputs(1, 64, 64, 8 * 100 + 4, seed=1))     # V not a multiple of 8
    ctx.force_path(binding.PATH_STREAM)
    with pytest.raises(binding.SlimSpecError) as e:
        ctx.slimspec_head_topk(x["h"], x["A"], x["B"], 4)
    assert e.value.status == binding.ERR_ALIGN
    ctx.force_path(binding.PATH_AUTO)
    ctx.slimspec_head_topk(x["h"], x["A"], x["B"], 4)
    assert ctx.last_path() == binding.PATH_GENERIC


# ---------------------------------------------------------------- the workloads

def _config_case(ctx, name, M, rows=None, path=binding.PATH_AUTO):
    c = synth.CONFIGS[name]
    x = synth.make_inputs(M, c.d, c.r, c.V, seed=c.seed, logit_scale=c.logit_scale)
    ids, lp = run_topk(ctx, x, c.k, path) if path != binding.PATH_AUTO else _auto(ctx, x, c.k)
    b = obits(x)
    hb = b["h"] if rows is None else b["h"][rows]
    ref = oracle.head_topk(hb, b["A"], b["B"], c.k)
    return check_topk(ref, ids, lp, rows=rows), ids, lp


def _auto(ctx, x, k):
    ctx.force_path(binding.PATH_AUTO)
    g = dev(x)
    ids, lp = ctx.slimspec_head_topk(g["h"], g["A"], g["B"], k)
    torch.cuda.synchronize()
    assert ctx.last_error() == binding.OK
    return ids.cpu().numpy(), lp.cpu().numpy()


@pytest.mark.parametrize("name,M", [("c0", 1), ("c1", 1), ("c1", 8), ("c2", 1), ("c2", 16)])
def test_workload_configs(ctx, name, M):
    st, _, _ = _config_case(ctx, name, M)
    assert st["rows"] == M
    assert st["max_lp_err"] <= LOGPROB_TOL


def test_throughput_batch_sampled_rows(ctx):
    # M = 512: the oracle checks rows at every position class of a 128-row tile plus seeded extras
    M = 512
    rng = np.random.default_rng(0)
    rows = sorted(set([0, 1, 63, 64, 127, 128, M // 2, M - 2, M - 1]) | set(rng.integers(0, M, 8).tolist()))
    st, ids, lp = _config_case(ctx, "c3", M, rows=rows)
    assert st["max_lp_err"] <= LOGPROB_TOL
    # rows the oracle did not see: a row's result must not depend on the batch around it
    c = synth.CONFIGS["c3"]
    x = synth.make_inputs(M, c.d, c.r, c.V, seed=c.seed)
    g = dev(x)
    # (a sub-batch that takes the same kernels in the same precision mode -- more than 256 rows --
    # but puts every row at another position of another 128-row tile)
    m0 = 200
    i1, l1 = ctx.slimspec_head_topk(g["h"][m0:].contiguous(), g["A"], g["B"], c.k)
    torch.cuda.synchronize()
    assert ctx.last_path() == binding.PATH_TENSOR
    i1, l1 = i1.cpu().numpy(), l1.cpu().numpy()
    for m in (200, 300, 383, 384, 509, 511):
        assert np.array_equal(i1[m - m0], ids[m])
        assert np.max(np.abs(l1[m - m0] - lp[m])) < 2e-4


@pytest.mark.parametrize("r,M", [(1024, 64), (2048, 4)])
def test_sweep_shapes_sampled_rows(r, M):
    # d = 8192 heads of the rank sweep: K too long for a resident code / X, several z chunks
    d, V, k = synth.SWEEP_D, synth.SWEEP_V, 10
    c = binding.Context(max_M=M, max_d=d, max_V=V, max_k=16)
    x = synth.make_inputs(M, d, r, V, seed=7)
    g = dev(x)
    ids, lp = c.slimspec_head_topk(g["h"], g["A"], g["B"], k)
    torch.cuda.synchronize()
    assert c.last_error() == binding.OK
    rows = sorted({0, M // 2, M - 1})
    b = obits(x)
    ref = oracle.head_topk(b["h"][rows], b["A"], b["B"], k)
    st = check_topk(ref, ids.cpu().numpy(), lp.cpu().numpy(), rows=rows)
    assert st["max_lp_err"] <= LOGPROB_TOL
    c.close()


# ---------------------------------------------------------------- full-rank baseline, logits

@pytest.mark.parametrize("M", [1, 8])
def test_fullhead_baseline(ctx, M):
    c = synth.CONFIGS["c1"]
    h = synth.make_h(M, c.d, c.seed)
    W = synth.make_W(c.d, c.V, c.seed)
    ctx.force_path(binding.PATH_AUTO)
    ids, lp = ctx.fullhead_topk(h.to(DEV), W.to(DEV), c.k)
    torch.cuda.synchronize()
    assert ctx.last_error() == binding.OK
    ref = oracle.fullhead_topk(oracle.bf16_bits(h), oracle.bf16_bits(W), c.k)
    st = check_topk(ref, ids.cpu().numpy(), lp.cpu().numpy())
    assert st["max_lp_err"] <= LOGPROB_TOL


def test_identity_downprojection_equals_fullhead_on_gpu(ctx):
    d, V, M, k = 128, 8 * 1234, 3, 10
    h = synth.make_h(M, d, 3)
    B = synth.make_B(d, V, 3)
    eye = torch.eye(d, dtype=torch.bfloat16)
    for path in (binding.PATH_GENERIC, binding.PATH_STREAM):
        ctx.force_path(path)
        i1, l1 = ctx.slimspec_head_topk(h.to(DEV), eye.to(DEV), B.to(DEV), k)
        i2, l2 = ctx.fullhead_topk(h.to(DEV), B.to(DEV), k)
        assert torch.equal(i1, i2)
        assert torch.max(torch.abs(l1 - l2)).item() < 1e-5


@pytest.mark.parametrize("path", [binding.PATH_GENERIC, binding.PATH_STREAM])
@pytest.mark.parametrize("M,d,r,V", [(1, 2048, 256, 128256), (6, 512, 128, 8 * 3001)])
def test_head_logits(ctx, path, M, d, r, V):
    x = synth.make_inputs(M, d, r, V, seed=2)
    g = dev(x)
    ctx.force_path(path)
    # canaries around the output catch writes out of bounds
    buf = torch.full((M * V + 512,), 12345.0, dtype=torch.float32, device=DEV)
    out = buf[256:256 + M * V].view(M, V)
    ctx.slimspec_head_logits(g["h"], g["A"], g["B"], out_logits=out)
    torch.cuda.synchronize()
    assert ctx.last_error() == binding.OK
    assert torch.all(buf[:256] == 12345.0) and torch.all(buf[256 + M * V:] == 12345.0)
    b = obits(x)
    ref = oracle.slimspec_logits(b["h"], b["A"], b["B"])
    assert np.max(np.abs(out.cpu().numpy().astype(np.float64) - ref)) <= 2e-2


def test_topk_outputs_do_not_overrun(ctx):
    M, d, r, V, k = 5, 256, 64, 8 * 999, 10
    g = dev(synth.make_inputs(M, d, r, V, seed=4))
    for path in (binding.PATH_GENERIC, binding.PATH_STREAM):
        ctx.force_path(path)
        ib = torch.full((M * k + 64,), -7, dtype=torch.int32, device=DEV)
        lb = torch.full((M * k + 64,), -7.0, dtype=torch.float32, device=DEV)
        ctx.slimspec_head_topk(g["h"], g["A"], g["B"], k, out_ids=ib[32:32 + M * k].view(M, k),
                               out_logprobs=lb[32:32 + M * k].view(M, k))
        torch.cuda.synchronize()
        assert torch.all(ib[:32] == -7) and torch.all(ib[32 + M * k:] == -7)
        assert torch.all(lb[:32] == -7.0) and torch.all(lb[32 + M * k:] == -7.0)
        assert torch.all(ib[32:32 + M * k] >= 0)


def test_planted_ties_resolve_to_lower_id(ctx):
    M, d, r, V, k = 2, 128, 64, 8 * 600, 6
    x = synth.make_inputs(M, d, r, V, seed=8)
    b = obits(x)
    best = int(np.argmax(oracle.slimspec_logits(b["h"], b["A"], b["B"])[0]))
    twin = (best + 2417) % V                      # lands in another slab
    x["B"][:, twin] = x["B"][:, best]
    for path in (binding.PATH_GENERIC, binding.PATH_STREAM):
        ids, lp = run_topk(ctx, x, k, path)
        assert ids[0, :2].tolist() == sorted([best, twin])
        assert lp[0, 0] == lp[0, 1]


def test_host_buffer_entry_point(ctx):
    c = synth.CONFIGS["c0"]
    x = synth.make_inputs(1, c.d, c.r, c.V, seed=c.seed)
    g = dev(x)
    ctx.force_path(binding.PATH_AUTO)
    ids_d, lp_d = ctx.slimspec_head_topk(g["h"], g["A"], g["B"], c.k)
    ids_h, lp_h = ctx.slimspec_head_topk_host(x["h"].pin_memory(), g["A"], g["B"], c.k)
    assert torch.equal(ids_d.cpu(), ids_h) and torch.equal(lp_d.cpu(), lp_h)


def test_argument_errors_launch_nothing(ctx):
    g = dev(synth.make_inputs(2, 64, 64, 800, seed=1))
    n0 = ctx.launch_count()
    lib = binding.load()
    import ctypes
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    ids = torch.empty((2, 4), dtype=torch.int32, device=DEV)
    lp = torch.empty((2, 4), dtype=torch.float32, device=DEV)
    call = lambda M, d, r, V, k, h=g["h"]: lib.slimspec_head_topk(
        ctx._h, p(h) if h is not None else None, p(g["A"]), p(g["B"]), M, d, r, V, k, p(ids), p(lp), None)
    assert call(2, 64, 64, 800, 4, h=None) == binding.ERR_NULL
    assert call(0, 64, 64, 800, 4) == binding.ERR_DIM
    assert call(2, 64, 64, 800, 0) == binding.ERR_DIM
    assert call(2, 64, 64, 800, 801) == binding.ERR_DIM
    assert call(2, 64, 64, 800, 65) == binding.ERR_DIM
    assert call(513, 64, 64, 800, 4) == binding.ERR_DIM
    assert call(2, 64, 64, 200008, 4) == binding.ERR_DIM
    assert ctx.launch_count() == n0


# ---------------------------------------------------------------- calls in a row, no host synchronisation

@pytest.mark.parametrize("M", [1, 3, 12])
def test_back_to_back_calls_keep_stream_order(ctx, M):
    """Kernels of one call are launched early behind the kernels of the call before (and behind
    whatever else precedes them in the stream).  Calls in a row, with no host synchronisation,
    alternate between two different inputs whose h is written by another kernel on the same stream
    just before each call; every result must equal that of the same call made alone.  (Two hundred
    calls: a race between the kernels of neighbouring calls need not show in the first few.)"""
    ctx.force_path(binding.PATH_AUTO)
    d, r, V, k = 1024, 128, 32 * 1024, 10
    xs = [dev(synth.make_inputs(M, d, r, V, seed=71 + i)) for i in range(2)]
    alone = []
    for x in xs:
        ids, lp = ctx.slimspec_head_topk(x["h"], x["A"], x["B"], k)
        torch.cuda.synchronize()
        alone.append((ids.clone(), lp.clone()))
    n = 200
    out_ids = [torch.full((M, k), -7, dtype=torch.int32, device=DEV) for _ in range(n)]
    out_lp = [torch.zeros((M, k), dtype=torch.float32, device=DEV) for _ in range(n)]
    hbuf = torch.zeros_like(xs[0]["h"])
    for i in range(n):
        x = xs[i % 2]
        hbuf.copy_(x["h"])            # a kernel on the same stream writes the call's input
        ctx.slimspec_head_topk(hbuf, x["A"], x["B"], k, out_ids=out_ids[i], out_logprobs=out_lp[i])
    torch.cuda.synchronize()
    assert ctx.last_error() == binding.OK
    for i in range(n):
        ids, lp = alone[i % 2]
        assert torch.equal(out_ids[i], ids), "call %d" % i
        assert torch.equal(out_lp[i], lp), "call %d" % i


# ---------------------------------------------------------------- large batches: oracle on sampled rows

def sampled_rows(M, extra=8, seed=0):
    """Rows at every position class of a 128-row tile, the ends, the middle, plus seeded extras."""
    rng = np.random.default_rng(seed)
    base = {0, 1, 63, 64, 127, 128, M // 2, M - 2, M - 1}
    return sorted({m for m in base if 0 <= m < M} | set(rng.integers(0, M, extra).tolist()))


@pytest.fixture(scope="module")
def big_ctx():
    c = binding.Context(max_M=1024, max_d=8192, max_V=160000, max_k=16)
    yield c
    c.close()


def test_fullhead_throughput_batch_sampled_rows(big_ctx):
    """The standard head at the throughput batch (M = 512, d = 4096): K is too long for a resident
    row block, so the activations go through their own ring next to the weight ring."""
    c = synth.CONFIGS["c3"]
    M = 512
    h = synth.make_h(M, c.d, c.seed)
    W = synth.make_W(c.d, c.V, c.seed)
    big_ctx.force_path(binding.PATH_AUTO)
    ids, lp = big_ctx.fullhead_topk(h.to(DEV), W.to(DEV), c.k)
    torch.cuda.synchronize()
    assert big_ctx.last_error() == binding.OK and big_ctx.last_path() == binding.PATH_TENSOR
    rows = sampled_rows(M)
    ref = oracle.fullhead_topk(oracle.bf16_bits(h)[rows], oracle.bf16_bits(W), c.k)
    st = check_topk(ref, ids.cpu().numpy(), lp.cpu().numpy(), rows=rows)
    assert st["max_lp_err"] <= 1e-3        # h is exact in bf16: only fp32 accumulation differs


@pytest.mark.parametrize("r,M", [(2048, 256), (512, 1024), (512, 256)])
def test_sweep_large_batches_sampled_rows(big_ctx, r, M):
    """d = 8192 heads of the rank sweep with several row blocks."""
    d, V, k = synth.SWEEP_D, synth.SWEEP_V, 10
    x = synth.make_inputs(M, d, r, V, seed=7)
    g = dev(x)
    big_ctx.force_path(binding.PATH_AUTO)
    ids, lp = big_ctx.slimspec_head_topk(g["h"], g["A"], g["B"], k)
    torch.cuda.synchronize()
    assert big_ctx.last_error() == binding.OK and big_ctx.last_path() == binding.PATH_TENSOR
    rows = sampled_rows(M, extra=4)
    b = obits(x)
    ref = oracle.head_topk(b["h"][rows], b["A"], b["B"], k)
    st = check_topk(ref, ids.cpu().numpy(), lp.cpu().numpy(), rows=rows)
    assert st["max_lp_err"] <= LOGPROB_TOL


def test_sweep_fullhead_largest_batch_sampled_rows(big_ctx):
    """Full rank at d = 8192, M = 1024: eight row blocks, 128 K chunks per tile."""
    d, V, k, M = synth.SWEEP_D, synth.SWEEP_V, 10, 1024
    h = synth.make_h(M, d, 7)
    W = synth.make_W(d, V, 7)
    big_ctx.force_path(binding.PATH_AUTO)
    ids, lp = big_ctx.fullhead_topk(h.to(DEV), W.to(DEV), k)
    torch.cuda.synchronize()
    assert big_ctx.last_error() == binding.OK and big_ctx.last_path() == binding.PATH_TENSOR
    rows = sampled_rows(M, extra=2)
    ref = oracle.fullhead_topk(oracle.bf16_bits(h)[rows], oracle.bf16_bits(W), k)
    st = check_topk(ref, ids.cpu().numpy(), lp.cpu().numpy(), rows=rows)
    assert st["max_lp_err"] <= 2e-3


@pytest.mark.parametrize("M", [16, 128])
def test_sharpened_logits_keep_the_logit_bound(big_ctx, M):
    """Logits scaled by four (the larger-vocabulary workload) at batch sizes where the code z is a
    tensor-core operand: raw logits must still lie within 2e-2 of the oracle's, which a code
    rounded once to bf16 would miss."""
    c = synth.CONFIGS["c2"]
    x = synth.make_inputs(M, c.d, c.r, c.V, seed=c.seed, logit_scale=c.logit_scale)
    g = dev(x)
    big_ctx.force_path(binding.PATH_AUTO)
    out = big_ctx.slimspec_head_logits(g["h"], g["A"], g["B"])
    ids, lp = big_ctx.slimspec_head_topk(g["h"], g["A"], g["B"], c.k)
    torch.cuda.synchronize()
    assert big_ctx.last_error() == binding.OK
    rows = sampled_rows(M, extra=2)
    b = obits(x)
    ref = oracle.head_topk(b["h"][rows], b["A"], b["B"], c.k)
    err = np.max(np.abs(out.cpu().numpy()[rows].astype(np.float64) - ref["logits"]))
    assert err <= 2e-2, "logit error %.3e" % err
    st = check_topk(ref, ids.cpu().numpy(), lp.cpu().numpy(), rows=rows)
    assert st["max_lp_err"] <= LOGPROB_TOL
