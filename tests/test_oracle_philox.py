"""Pins of the oracle's Philox4x32-10: published known answers and uniformity."""
import os

import numpy as np
import scipy.stats

from oracle import philox

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox_kat.txt")


def test_known_answers():
    rows = [l.split() for l in open(GOLD) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        assert philox.philox4x32_10(w[0:4], w[4:6]) == tuple(w[6:10])


def test_uniforms_are_uniform():
    u = np.array([philox.uniform(12345, 0, b, n, s) for b in range(4) for n in range(500) for s in (0, 1)])
    assert u.min() >= 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 0.02
    assert scipy.stats.kstest(u, "uniform").pvalue > 1e-3
    assert len(np.unique(u)) > 0.99 * len(u)


def test_streams_differ():
    a = philox.uniform(7, 0, 0, 5, 0)
    assert a != philox.uniform(7, 0, 0, 5, 1)
    assert a != philox.uniform(7, 1, 0, 5, 0)
    assert a != philox.uniform(8, 0, 0, 5, 0)
    assert a != philox.uniform(7 + (1 << 32), 0, 0, 5, 0)     # high key word is used
    assert a == philox.uniform(7, 0, 0, 5, 0)
