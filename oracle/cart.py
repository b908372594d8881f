"""Oracle: training of the entropy stratifier (test infrastructure only).

Sec. 4.2 of the paper: a 3-layer CART regression tree on one feature, x = Phi(P*) (cumulative
meta-path Top-K entropy), with the Terminal Confidence Rank y as the target.  A split threshold s
cuts a node's samples D into D_left = {x < s} and D_right = {x >= s}; Eq. 2 scores it by

    L(s) = sum over j in {left, right} of  |D_j| / |D|  *  sum over D_j of (y - mu_j)^2

with mu_j the mean rank of the part, and the split with the smallest L is taken.  Applied
recursively three times this gives 8 bins, i.e. 7 ascending thresholds.  Candidate thresholds
are the midpoints between consecutive distinct feature values (the usual CART convention; the
paper does not say), ties in L go to the smallest threshold.

App. A.4: the low-entropy sample sets of trees of different depth are compared by the Jaccard
coefficient |A and B| / |A or B|, the low-entropy region being the lowest 3/8 of the bins at
every depth ("equivalent proportional selection").

Everything is the plain definition: every candidate split is scored by summing over the samples.
"""

import numpy as np


def split_loss(x, y, s):
    """Eq. 2 for threshold s on the samples (x, y)."""
    x, y = np.asarray(x, dtype=np.float64), np.asarray(y, dtype=np.float64)
    total = 0.0
    for part in (y[x < s], y[x >= s]):
        if len(part):
            total += len(part) / len(y) * float(((part - part.mean()) ** 2).sum())
    return total


def best_split(x, y):
    """(threshold, loss) of the best split of one node, or None if all feature values are equal."""
    xs = np.unique(np.asarray(x, dtype=np.float64))
    best = None
    for a, b in zip(xs[:-1], xs[1:]):
        s = 0.5 * (a + b)
        l = split_loss(x, y, s)
        if best is None or l < best[1]:
            best = (s, l)
    return best


def fit_thresholds(x, y, depth=3):
    """The 2^depth - 1 thresholds of the tree, ascending.  A node that cannot be split (one distinct
    feature value) raises ValueError."""
    x, y = np.asarray(x, dtype=np.float64), np.asarray(y, dtype=np.float64)
    nodes = [(-np.inf, np.inf)]
    thresholds = []
    for _ in range(depth):
        nxt = []
        for lo, hi in nodes:
            sel = (x >= lo) & (x < hi)
            sp = best_split(x[sel], y[sel])
            if sp is None:
                raise ValueError("a node holds a single feature value")
            thresholds.append(sp[0])
            nxt += [(lo, sp[0]), (sp[0], hi)]
        nodes = nxt
    return sorted(thresholds)


def bins_of(x, thresholds):
    """bin = number of thresholds <= x (the lookup the verification step uses)."""
    return np.searchsorted(np.asarray(thresholds, dtype=np.float64), np.asarray(x, dtype=np.float64), side="right")


def low_entropy_set(x, thresholds):
    """Indices of the samples in the lowest 3/8 of the bins of a tree with len(thresholds) + 1 bins."""
    n_bins = len(thresholds) + 1
    return set(np.nonzero(bins_of(x, thresholds) < 3 * n_bins // 8)[0].tolist())


def jaccard(a, b):
    a, b = set(a), set(b)
    return len(a & b) / len(a | b) if (a | b) else 1.0
