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


def test_offset_high_word_selects_another_stream():
    """Counter convention of the acceptance step: (offset low word, b, node, stream + 2 * offset high word)."""
    seed = 0x0123456789ABCDEF
    key = (seed & 0xFFFFFFFF, seed >> 32)
    for off, b, node, stream in ((0, 0, 0, 0), (7, 3, 5, 1), ((9 << 32) + 7, 3, 5, 1), ((1 << 63) - 1, 4095, 127, 0)):
        words = philox.philox4x32_10((off & 0xFFFFFFFF, b, node, stream + 2 * (off >> 32)), key)
        assert philox.uniform(seed, off, b, node, stream) == (words[0] >> 8) * 2.0 ** -24
    assert philox.uniform(seed, 7, 3, 5, 1) != philox.uniform(seed, (1 << 32) + 7, 3, 5, 1)
