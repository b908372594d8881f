"""Pins of the stratifier-training oracle (Sec. 4.2, Eq. 2; App. A.4): hand-evaluated losses, recovery of planted
steps, agreement with scikit-learn's CART where Eq. 2 and the plain squared-error criterion coincide, invariances."""
import os

import numpy as np
import pytest
from sklearn.tree import DecisionTreeRegressor

from oracle import cart

GOLD = os.path.join(os.path.dirname(__file__), "golden", "cart_eq2.txt")


def test_eq2_hand_evaluated_losses_and_best_split():
    rows = [l.split("|") for l in open(GOLD) if l.strip() and not l.startswith("#")]
    for xs, ys, s, want in rows:
        x = [float(v) for v in xs.split(",")]
        y = [float(v) for v in ys.split(",")]
        assert cart.split_loss(x, y, float(s)) == pytest.approx(float(want), rel=1e-9)
    assert cart.best_split([1, 2, 3, 4], [0, 0, 3, 5]) == (2.5, pytest.approx(1.0))
    assert cart.best_split([1, 2, 3, 4, 5, 6], [0, 4, 4, 4, 4, 10])[0] == 5.5
    assert cart.best_split([3, 3, 3], [1, 2, 3]) is None


def test_planted_steps_are_recovered():
    """Eight plateaus of the target at known feature boundaries: the seven thresholds are the midpoints."""
    rng = np.random.default_rng(0)
    edges = np.array([0.0, 1.0, 2.5, 3.0, 4.5, 6.0, 6.5, 8.0, 9.0])
    # heights with a hierarchy of jumps (100 between the halves, 10 between the quarters, 1 between neighbours), so
    # that the greedy splits halve the plateaus at every layer
    levels = np.array([100 * (i >> 2) + 10 * ((i >> 1) & 1) + (i & 1) for i in range(8)], dtype=np.float64)
    x = np.concatenate([rng.uniform(edges[i] + 0.1, edges[i + 1] - 0.1, 40) for i in range(8)])
    y = np.concatenate([np.full(40, levels[i]) for i in range(8)])
    th = cart.fit_thresholds(x, y, 3)
    xs = np.sort(x)
    want = [0.5 * (xs[40 * i - 1] + xs[40 * i]) for i in range(1, 8)]
    assert np.allclose(th, want, atol=1e-12)
    assert cart.bins_of(x, th).tolist() == np.repeat(np.arange(8), 40).tolist()


@pytest.mark.parametrize("seed", range(3))
def test_agrees_with_sklearn_on_balanced_step_data(seed):
    """Eq. 2 weights a part's squared error by its share of the node; scikit-learn's criterion is the unweighted
    sum.  On noise-free plateaus of equal size with a hierarchy of jumps both pick the planted boundaries (every
    best split halves its node, where the two criteria differ by a constant factor), so the trees agree."""
    rng = np.random.default_rng(seed)
    x = np.sort(rng.uniform(0, 10, 256))
    sg = rng.choice([-1.0, 1.0], 3)
    y = np.repeat([sg[2] * 100 * (i >> 2) + sg[1] * 10 * ((i >> 1) & 1) + sg[0] * (i & 1) for i in range(8)], 32)
    th = cart.fit_thresholds(x, y, 3)
    sk = DecisionTreeRegressor(max_depth=3).fit(x[:, None], y)
    sk_th = sorted(t for t, f in zip(sk.tree_.threshold, sk.tree_.feature) if f >= 0)
    assert np.allclose(th, sk_th, atol=1e-9)


def test_invariances_and_optimality():
    rng = np.random.default_rng(5)
    x = rng.uniform(0, 8, 120)
    y = np.round(3 * x + rng.normal(0, 4, 120))
    s, l = cart.best_split(x, y)
    xs = np.unique(x)
    assert all(l <= cart.split_loss(x, y, 0.5 * (a + b)) + 1e-12 for a, b in zip(xs[:-1], xs[1:]))
    th = cart.fit_thresholds(x, y, 3)
    assert len(th) == 7 and all(a < b for a, b in zip(th[:-1], th[1:]))
    assert np.allclose(cart.fit_thresholds(x, y + 100.0, 3), th)            # the target's offset does not matter
    assert np.allclose(cart.fit_thresholds(2.0 * x + 1.0, y, 3), 2.0 * np.array(th) + 1.0)
    with pytest.raises(ValueError):
        cart.fit_thresholds(np.ones(10), np.arange(10.0), 3)


def test_jaccard_and_low_entropy_sets():
    assert cart.jaccard({1, 2, 3}, {2, 3, 4}) == 0.5 and cart.jaccard(set(), set()) == 1.0
    x = np.arange(16, dtype=np.float64)
    th8 = [1.5, 3.5, 5.5, 7.5, 9.5, 11.5, 13.5]              # 8 bins of two samples: the low set is bins 0..2
    assert cart.low_entropy_set(x, th8) == set(range(6))
    th16 = list(np.arange(0.5, 15, 1.0))                     # 16 bins of one sample: the low set is bins 0..5
    assert cart.low_entropy_set(x, th16) == set(range(6))
    assert cart.jaccard(cart.low_entropy_set(x, th8), cart.low_entropy_set(x, th16)) == 1.0
