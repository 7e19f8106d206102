"""Comparison rules between the CUDA library's results and the CPU oracle's.

Floating point: log-probs and logits within 2e-2 absolute (bf16 weights, fp32 accumulation).
Top-k ids: where the oracle's gap between ranks k and k+1 exceeds 4e-2 the id SET must be the
oracle's, and position j must hold the oracle's id wherever the oracle's logit at rank j is
more than 4e-2 away from both neighbours; elsewhere the answer must be a valid top-k under
that tolerance (nothing clearly better left out, nothing clearly worse included).
"""
from __future__ import annotations

import numpy as np

LOGPROB_TOL = 2e-2
GAP_TOL = 4e-2


def check_topk(ref: dict, ids, logprobs, rows=None, lp_tol: float = LOGPROB_TOL, gap_tol: float = GAP_TOL):
    """ref: oracle.head_topk(...) result for the rows in `rows` (default: all, in order).

    ids / logprobs: the library's outputs for ALL rows (numpy).  Returns statistics;
    raises AssertionError on the first violated rule."""
    ids = np.asarray(ids)
    logprobs = np.asarray(logprobs, dtype=np.float64)
    M_ref, V = ref["logits"].shape
    rows = list(range(M_ref)) if rows is None else list(rows)
    k = ids.shape[1]
    assert ref["ids"].shape[1] == k
    stats = {"rows": len(rows), "exact_rows": 0, "tolerant_rows": 0, "max_lp_err": 0.0, "order_identical": 0}
    for n, m in enumerate(rows):
        logit = ref["logits"][n]
        lse = ref["lse"][n]
        got = ids[m].astype(np.int64)
        assert got.min() >= 0 and got.max() < V, "row %d: id out of range" % m
        assert len(set(got.tolist())) == k, "row %d: duplicate ids %s" % (m, got)
        # log-prob of the returned id against the oracle's log-prob of that same id
        err = np.abs(logprobs[m] - (logit[got] - lse))
        stats["max_lp_err"] = max(stats["max_lp_err"], float(err.max()))
        assert err.max() <= lp_tol, "row %d: log-prob error %.3e > %.1e" % (m, err.max(), lp_tol)
        # the library's own values must be sorted
        assert np.all(np.diff(logprobs[m]) <= 0), "row %d: returned log-probs not non-increasing" % m
        top = ref["top_logits"][n]
        kth, nxt = top[k - 1], ref["next_logit"][n]
        want = ref["ids"][n].astype(np.int64)
        if kth - nxt > gap_tol:
            assert set(got.tolist()) == set(want.tolist()), "row %d: id set differs from the oracle's" % m
            stats["exact_rows"] += 1
            ext = np.concatenate(([np.inf], top, [nxt]))
            for j in range(k):
                if ext[j] - ext[j + 1] > gap_tol and ext[j + 1] - ext[j + 2] > gap_tol:
                    assert got[j] == want[j], "row %d: rank %d holds %d, oracle %d" % (m, j, got[j], want[j])
        else:
            stats["tolerant_rows"] += 1
            must = np.nonzero(logit > kth + gap_tol)[0]
            assert set(must.tolist()) <= set(got.tolist()), "row %d: a clearly better token was left out" % m
            assert logit[got].min() >= kth - gap_tol, "row %d: a clearly worse token was returned" % m
        # order under tolerance: oracle logits of the returned ids never rise by more than the tolerance
        assert np.all(np.diff(logit[got]) <= gap_tol), "row %d: order violates the oracle's by > tol" % m
        if np.array_equal(got, want):
            stats["order_identical"] += 1
    return stats
