"""The byte and flop counters behind every roofline fraction of bench.py, against the cost
ratio of Section 4.1: the low-rank head costs (r d + V r) / (V d) = (r / d)(1 + d / V) of the
standard head, in weights read and in multiply-adds."""
import itertools

import pytest

import bench


@pytest.mark.parametrize("d,r,V", [(2048, 256, 128256), (4096, 512, 128256), (5120, 640, 152064),
                                   (8192, 512, 128256), (8192, 2048, 128256), (8, 2, 37)])
def test_cost_ratio_closed_form(d, r, V):
    closed = (r / d) * (1.0 + d / V)
    # flops: 2 M (d r + r V) against 2 M d V, for any M
    for M in (1, 8, 512):
        assert bench.head_flops(M, d, r, V) / bench.fullhead_flops(M, d, V) == pytest.approx(closed, rel=1e-12)
    # weight bytes: what is left of the byte counters once activations and outputs are taken out
    M, k = 1, 10
    w_low = bench.head_bytes(M, d, r, V, k) - 2 * M * d - 8 * M * k
    w_full = bench.fullhead_bytes(M, d, V, k) - 2 * M * d - 8 * M * k
    assert w_low == 2 * (d * r + r * V) and w_full == 2 * d * V
    assert w_low / w_full == pytest.approx(closed, rel=1e-12)


def test_counters_by_hand():
    # d=4, r=2, V=8, M=3, k=1: A 8 + B 16 weights, bf16; h 12 elements; 3 ids + 3 log-probs
    assert bench.head_bytes(3, 4, 2, 8, 1) == 2 * 24 + 2 * 12 + 8 * 3
    assert bench.head_flops(3, 4, 2, 8) == 2 * 3 * 24
    assert bench.fullhead_bytes(3, 4, 8, 1) == 2 * 32 + 2 * 12 + 8 * 3
    assert bench.fullhead_flops(3, 4, 8) == 2 * 3 * 32


def test_speedup_target_is_the_inverse_ratio():
    d, r, V = 4096, 512, 128256
    assert bench.bytes_ratio_target(d, r, V) == pytest.approx(0.8 / ((r / d) * (1 + d / V)), rel=1e-12)
    assert bench.bytes_ratio_target(d, r, V) == pytest.approx(6.2, abs=0.02)
