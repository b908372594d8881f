"""Pins of the oracle's row statistics: closed forms, invariances, a hand-worked row and an
independent library (scipy)."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import row_stats as rs


def test_constant_row_closed_forms():
    V, K, c = 1000, 10, 3.25
    s = rs.row_stats(np.full(V, c), K)
    assert s["H"] == pytest.approx(math.log(V), rel=1e-12)
    assert s["I_topk"] == pytest.approx(math.log(K), rel=1e-12)
    assert s["I_trunc"] == pytest.approx(K / V * math.log(V), rel=1e-12)
    assert s["lse"] == pytest.approx(c + math.log(V), rel=1e-12)
    assert s["max"] == c
    assert list(s["topk_idx"]) == list(range(K))          # ties: lowest index first


def test_one_hot_and_two_point():
    row = np.full(512, -1e4); row[77] = 2.0
    s = rs.row_stats(row, 10)
    assert s["H"] == 0.0 and s["I_topk"] == 0.0 and s["I_trunc"] == 0.0
    assert s["topk_idx"][0] == 77 and s["lse"] == pytest.approx(2.0)
    row[300] = 2.0
    s = rs.row_stats(row, 10)
    assert s["H"] == pytest.approx(math.log(2), rel=1e-12)
    assert s["I_topk"] == pytest.approx(math.log(2), rel=1e-12)
    assert list(s["topk_idx"][:2]) == [77, 300]


def test_hand_worked_row():
    # logits ln 1..ln 4 -> p = (0.1, 0.2, 0.3, 0.4)
    row = np.log(np.array([1.0, 2.0, 3.0, 4.0]))
    s = rs.row_stats(row, 2)
    H = -(0.1 * math.log(0.1) + 0.2 * math.log(0.2) + 0.3 * math.log(0.3) + 0.4 * math.log(0.4))
    assert s["H"] == pytest.approx(H, rel=1e-12)
    assert list(s["topk_idx"]) == [3, 2]
    assert s["I_topk"] == pytest.approx(-(4 / 7 * math.log(4 / 7) + 3 / 7 * math.log(3 / 7)), rel=1e-12)
    assert s["I_trunc"] == pytest.approx(-(0.4 * math.log(0.4) + 0.3 * math.log(0.3)), rel=1e-12)
    assert s["lse"] == pytest.approx(math.log(10.0), rel=1e-12)


def test_shift_invariance_and_k_equals_v():
    rng = np.random.default_rng(1)
    row = rng.standard_normal(300) * 3
    a, b = rs.row_stats(row, 7), rs.row_stats(row + 11.5, 7)
    for key in ("H", "I_topk", "I_trunc"):
        assert a[key] == pytest.approx(b[key], rel=1e-10)
    assert b["lse"] - a["lse"] == pytest.approx(11.5, rel=1e-12)
    assert list(a["topk_idx"]) == list(b["topk_idx"])
    full = rs.row_stats(row, 300)
    assert full["I_topk"] == pytest.approx(full["H"], rel=1e-12)
    assert full["I_trunc"] == pytest.approx(full["H"], rel=1e-12)


def test_against_scipy():
    rng = np.random.default_rng(2)
    for scale in (0.2, 1.0, 4.0):
        row = rng.standard_normal(5000) * scale
        s = rs.row_stats(row, 10)
        p = scipy.special.softmax(row)
        assert s["H"] == pytest.approx(scipy.stats.entropy(p), rel=1e-10)
        assert s["lse"] == pytest.approx(scipy.special.logsumexp(row), rel=1e-12)
        top = np.sort(p)[::-1][:10]
        assert s["I_topk"] == pytest.approx(scipy.stats.entropy(top / top.sum()), rel=1e-10)
        assert s["I_topk"] <= math.log(10) + 1e-12


def test_topk_order_with_planted_ties():
    row = np.zeros(64); row[[5, 9, 40]] = 2.0; row[[3, 50]] = 1.0
    idx = rs.topk_indices(row, 6)
    assert list(idx) == [5, 9, 40, 3, 50, 0]
