"""Oracle step 1: per-row vocabulary statistics (test infrastructure only).

Follows the inner sum of Eq. 1 (Sec. 4.1): for one next-token distribution, the
entropy of the normalised probabilities of its Top-K tokens.  Everything is the
textbook two-pass definition in float64.
"""

import numpy as np


def softmax64(row):
    """p = softmax(row) by the two-pass definition; returns (p, max, log-sum-exp)."""
    x = np.asarray(row, dtype=np.float64)
    m = x.max()
    e = np.exp(x - m)
    s = e.sum()
    return e / s, m, m + np.log(s)


def xlogx_sum(p):
    """-sum p ln p with the convention 0 ln 0 = 0 (nats)."""
    p = np.asarray(p, dtype=np.float64)
    nz = p > 0
    return float(-(p[nz] * np.log(p[nz])).sum())


def topk_indices(row, k):
    """Indices of the k largest logits, ordered by (value descending, index ascending)."""
    x = np.asarray(row, dtype=np.float64)
    order = np.lexsort((np.arange(x.shape[0]), -x))
    return order[:k]


def row_stats(row, k):
    """Statistics of one logits row.

    Returns dict with
      max, lse      row maximum and log-sum-exp
      H             Shannon entropy of softmax(row), nats
      topk_idx/val  the K largest logits (ties: lowest index first)
      I_topk        entropy of the Top-K probabilities renormalised to sum 1
                    (Eq. 1 inner sum, "normalized probabilities of the Top-K tokens")
      I_trunc       -sum over the Top-K of p ln p with p the vocabulary-wide softmax
                    (the other reading of "normalized")
    """
    p, m, lse = softmax64(row)
    idx = topk_indices(row, k)
    pk = p[idx]
    ptilde = pk / pk.sum()
    return dict(max=float(m), lse=float(lse), H=xlogx_sum(p),
                topk_idx=idx.astype(np.int64), topk_val=np.asarray(row, dtype=np.float64)[idx],
                I_topk=xlogx_sum(ptilde), I_trunc=xlogx_sum(pk))


def batch_row_stats(logits, k):
    """row_stats for every row of a [rows, V] matrix; returns a dict of stacked arrays."""
    rows = [row_stats(r, k) for r in np.asarray(logits, dtype=np.float64)]
    return {key: np.stack([np.asarray(r[key]) for r in rows]) for key in rows[0]}
