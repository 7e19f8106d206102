"""Pins for the CPU oracle: each checks it against something other than itself.

Closed forms, a hand-worked example, brute force in another association order, library
routines (numpy matmul / lexsort, scipy log_softmax) and invariants of Section 4.1's
definition logits = W_up W_down h.
"""
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

import oracle
from paper_2605_10453_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "integer_head_example.txt")


def bits(x):
    """float array (values exactly representable in bf16) -> uint16 bf16 bits."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32))
    b = t.to(torch.bfloat16)
    assert torch.equal(b.to(torch.float32), t), "test value not exact in bf16"
    return oracle.bf16_bits(b)


def widen(u16):
    """uint16 bf16 bits -> float64 values, via numpy only."""
    return (u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rand_bits(shape, seed, std=1.0):
    g = torch.Generator().manual_seed(seed)
    return oracle.bf16_bits((torch.randn(shape, generator=g) * std).to(torch.bfloat16))


def load_golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        out.setdefault(key, []).append([float(v) for v in vals])
    return out


# ---------------------------------------------------------------- logits --------------

def test_hand_worked_integer_example():
    g = load_golden()
    h, A, B, W = (np.array(g[k]) for k in ("h", "A", "B", "W"))
    assert h.shape == (2, 4) and A.shape == (4, 2) and B.shape == (2, 5) and W.shape == (4, 5)
    z = oracle.downproj(bits(h), bits(A))
    assert np.array_equal(z, np.array(g["z"]))
    logits = oracle.slimspec_logits(bits(h), bits(A), bits(B))
    assert np.array_equal(logits, np.array(g["logits"]))
    assert np.array_equal(oracle.fullhead_logits(bits(h), bits(W)), np.array(g["logits"]))
    res = oracle.head_topk(bits(h), bits(A), bits(B), 3)
    assert np.array_equal(res["ids"], np.array(g["top3"], dtype=np.int32))
    want_lse = np.array(g["lse"]).ravel()
    assert np.allclose(res["lse"], want_lse, rtol=0, atol=1e-13)
    want_lp = np.take_along_axis(np.array(g["logits"]), res["ids"].astype(np.int64), 1) - want_lse[:, None]
    assert np.allclose(res["logprobs"], want_lp, rtol=0, atol=1e-13)


def test_identity_downprojection_is_the_standard_head():
    d, V, M = 16, 53, 3
    h = rand_bits((M, d), 1)
    B = rand_bits((d, V), 2, 0.25)
    eye = bits(np.eye(d))
    assert np.array_equal(oracle.slimspec_logits(h, eye, B), oracle.fullhead_logits(h, B))


def test_tiny_bruteforce_other_association():
    d, r, V, M = 8, 2, 37, 3
    h, A, B = rand_bits((M, d), 3), rand_bits((d, r), 4, 0.35), rand_bits((r, V), 5, 0.7)
    AB = np.zeros((d, V))
    for i in range(d):
        for v in range(V):
            AB[i, v] = math.fsum(widen(A)[i, j] * widen(B)[j, v] for j in range(r))
    want = np.zeros((M, V))
    for m in range(M):
        for v in range(V):
            want[m, v] = math.fsum(widen(h)[m, i] * AB[i, v] for i in range(d))
    got = oracle.slimspec_logits(h, A, B)
    assert np.max(np.abs(got - want)) <= 1e-12


@pytest.mark.parametrize("M,d,r,V", [(1, 8, 2, 37), (5, 24, 7, 130), (3, 64, 16, 1000)])
def test_against_numpy_matmul(M, d, r, V):
    h, A, B = rand_bits((M, d), 6), rand_bits((d, r), 7, d ** -0.5), rand_bits((r, V), 8, r ** -0.5)
    z = oracle.downproj(h, A)
    assert np.max(np.abs(z - widen(h) @ widen(A))) <= 1e-12
    got = oracle.slimspec_logits(h, A, B)
    assert np.max(np.abs(got - (widen(h) @ widen(A)) @ widen(B))) <= 1e-12
    W = rand_bits((d, V), 9, d ** -0.5)
    assert np.max(np.abs(oracle.fullhead_logits(h, W) - widen(h) @ widen(W))) <= 1e-12


def test_linearity_in_h_exact_on_integers():
    rng = np.random.default_rng(0)
    d, r, V = 12, 3, 41
    h1 = rng.integers(-4, 5, (2, d)).astype(np.float64)
    h2 = rng.integers(-4, 5, (2, d)).astype(np.float64)
    A = rng.integers(-3, 4, (d, r)).astype(np.float64)
    B = rng.integers(-3, 4, (r, V)).astype(np.float64)
    f = lambda h: oracle.slimspec_logits(bits(h), bits(A), bits(B))
    assert np.array_equal(f(h1 + h2), f(h1) + f(h2))
    assert np.array_equal(f(2 * h1), 2 * f(h1))
    assert np.array_equal(f(np.zeros_like(h1)), np.zeros((2, V)))


def test_rank_of_logit_matrix_at_most_r():
    M, d, r, V = 9, 20, 3, 64
    L = oracle.slimspec_logits(rand_bits((M, d), 10), rand_bits((d, r), 11, 0.3), rand_bits((r, V), 12, 0.5))
    s = np.linalg.svd(L, compute_uv=False)
    assert s[r - 1] > 1e-3 * s[0]
    assert s[r] <= 1e-12 * s[0]


def test_row_independence_and_thread_count():
    M, d, r, V = 6, 32, 8, 301
    h, A, B = rand_bits((M, d), 13), rand_bits((d, r), 14, 0.2), rand_bits((r, V), 15, 0.4)
    full = oracle.slimspec_logits(h, A, B)
    for m in (0, 3, 5):
        assert np.array_equal(oracle.slimspec_logits(h[m:m + 1], A, B)[0], full[m])
    n = oracle.threads()
    try:
        oracle.set_threads(1)
        assert np.array_equal(oracle.slimspec_logits(h, A, B), full)
    finally:
        oracle.set_threads(n)


def test_statistical_closed_form_at_full_vocabulary():
    # For B ~ N(0, 1/r) the logits of a row are N(0, |z|^2 / r), hence
    # lse ~ ln V + |z|^2 / (2 r) up to ~ sqrt((e^{s^2} - 1) / V)  (about 4e-3 at s = 1).
    c = synth.CONFIGS["c0"]
    x = synth.make_inputs(1, c.d, c.r, c.V, seed=c.seed)
    h, A, B = (oracle.bf16_bits(x[k]) for k in ("h", "A", "B"))
    z = widen(h) @ widen(A)
    s2 = float((z ** 2).sum()) / c.r
    res = oracle.head_topk(h, A, B, c.k)
    assert abs(res["lse"][0] - (math.log(c.V) + s2 / 2)) < 0.05
    assert abs(res["logits"].std() - math.sqrt(s2)) < 0.02 * math.sqrt(s2)


# ---------------------------------------------------------------- log-softmax ---------

def test_log_softmax_closed_forms():
    V = 1000
    lp, lse = oracle.log_softmax(np.full((1, V), 3.25))
    assert np.allclose(lp, -math.log(V), rtol=0, atol=1e-13) and abs(lse[0] - 3.25 - math.log(V)) < 1e-13
    # n_a entries equal a, n_b entries equal b: lse = a + log(n_a + n_b e^{b-a})
    row = np.array([[2.0] * 3 + [-1.0] * 7])
    lp, lse = oracle.log_softmax(row)
    assert abs(lse[0] - (2.0 + math.log(3 + 7 * math.exp(-3.0)))) < 1e-13
    # huge logits must not overflow
    lp, lse = oracle.log_softmax(np.array([[1000.0, 1000.0, -1000.0]]))
    assert abs(lse[0] - (1000.0 + math.log(2.0))) < 1e-12 and np.isfinite(lp).all()


def test_log_softmax_normalises_and_matches_library():
    rng = np.random.default_rng(1)
    x = rng.normal(0, 4, (7, 2500))
    lp, lse = oracle.log_softmax(x)
    assert np.max(np.abs(scipy.special.logsumexp(lp, axis=1))) <= 1e-12
    assert np.max(np.abs(lp - scipy.special.log_softmax(x, axis=1))) <= 1e-12
    lp2, lse2 = oracle.log_softmax(x + 17.0)
    assert np.max(np.abs(lp2 - lp)) <= 1e-12 and np.max(np.abs(lse2 - lse - 17.0)) <= 1e-12


def test_head_logprobs_sum_to_one():
    M, d, r, V = 4, 32, 8, 777
    res = oracle.head_topk(rand_bits((M, d), 16), rand_bits((d, r), 17, 0.2), rand_bits((r, V), 18, 1.0), 5)
    assert np.max(np.abs(scipy.special.logsumexp(res["logprob_full"], axis=1))) <= 1e-12
    picked = np.take_along_axis(res["logprob_full"], res["ids"].astype(np.int64), 1)
    assert np.array_equal(picked, res["logprobs"])


# ---------------------------------------------------------------- top-k ---------------

def full_sort_ids(row):
    return np.lexsort((np.arange(row.size), -row))   # value descending, then id ascending


def test_topk_is_prefix_of_full_sort():
    rng = np.random.default_rng(2)
    x = rng.normal(size=(5, 999))
    for k in (1, 2, 10, 64, 999):
        ids, vals, nxt = oracle.topk(x, k)
        for m in range(5):
            order = full_sort_ids(x[m])
            assert np.array_equal(ids[m], order[:k])
            assert np.array_equal(vals[m], x[m][order[:k]])
            assert nxt[m] == (x[m][order[k]] if k < 999 else -np.inf)
    assert np.array_equal(oracle.topk(x, 1)[0][:, 0], np.argmax(x, axis=1))
    assert np.array_equal(np.sort(oracle.topk(x, 999)[0], axis=1), np.tile(np.arange(999), (5, 1)))


def test_topk_ties_go_to_lower_id():
    x = np.array([[1.0, 5.0, 5.0, 0.0, 5.0, 7.0, 7.0, -1.0]])
    ids, vals, nxt = oracle.topk(x, 4)
    assert ids.tolist() == [[5, 6, 1, 2]] and vals.tolist() == [[7.0, 7.0, 5.0, 5.0]] and nxt[0] == 5.0
    # duplicate vocabulary columns of B give exactly equal logits
    d, r, V = 8, 4, 20
    h, A = rand_bits((1, d), 19), rand_bits((d, r), 20, 0.4)
    B = rand_bits((r, V), 21, 0.6)
    best = int(np.argmax(oracle.slimspec_logits(h, A, B)[0]))
    other = (best + 7) % V
    B[:, other] = B[:, best]
    res = oracle.head_topk(h, A, B, 2)
    assert res["ids"][0].tolist() == sorted([best, other])
    assert res["top_logits"][0, 0] == res["top_logits"][0, 1]


def test_topk_rejects_bad_k():
    with pytest.raises(ValueError):
        oracle.topk(np.zeros((1, 4)), 5)
    with pytest.raises(ValueError):
        oracle.topk(np.zeros((1, 4)), 0)
