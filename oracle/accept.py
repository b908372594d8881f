"""Oracle steps 6-7: lossless acceptance of the longest path (test infrastructure only).

Greedy (temperature 0, the paper's default setting, Sec. 5): a draft token is accepted
iff it equals the target model's argmax after its parent.  Sampling (Sec. 2.1): a draft
token x is accepted with probability min(1, p(x) / q(x)); on rejection the target
distribution is replaced by the normalised residual max(p - q, 0) and the next sibling
is tried (the chain rule of Sec. 2.1 applied to each sibling in turn, as in tree-based
verification); when no candidate is left the next token is drawn from the residual.

Deterministic proposals (a second reading of Sec. 2.1 for drafts that propose one fixed token per
candidate instead of a sample: the proposal distribution of candidate x is the point mass on its
token): the same chain rule with q = point mass, so x is accepted with probability r(token of x)
and a rejection removes that token from the residual.

Inputs use the pruned ("compact") tree: parent[i] < i, node 0 the root; target[i] is the
target model's logits row after kept node i, draft[i] the draft model's row after it.
"""

import numpy as np

from .row_stats import softmax64


def argmax_low(row):
    """Index of the maximum; ties go to the lowest index."""
    row = np.asarray(row)
    return int(np.nonzero(row == row.max())[0][0])


def children_of(parent, cur):
    return [i for i in range(len(parent)) if parent[i] == cur]


def greedy(parent, token, target):
    """Returns (path nodes incl. root, bonus token).  The walk starts at the root and moves to
    the child whose token equals the argmax of the current node's target row, until none does;
    the bonus token is the argmax at the node where the walk stops."""
    path = [0]
    cur = 0
    while True:
        g = argmax_low(target[cur])
        nxt = [c for c in children_of(parent, cur) if token[c] == g]
        if not nxt:
            return path, g
        cur = nxt[0]
        path.append(cur)


def rejection(parent, token, target, draft, temperature, u_accept, u_final, trace=None):
    """Multi-candidate rejection sampling down the tree.

    u_accept[i]: the uniform used for the accept test of kept node i; u_final: the uniform of
    the final draw.  At node cur with p = softmax(target[cur] / T), q = softmax(draft[cur] / T),
    r = p: children are tried in index order; child x is accepted iff u_accept[x] < min(1,
    r[tok] / q[tok]); otherwise r <- normalise(max(r - q, 0)).  After the last rejection (or at
    a leaf, where r = p) the bonus token is the smallest j with cumsum(r)[j] > u_final.
    ``trace`` (a list) receives (u, a) of every accept test and (u_final, cdf_below, cdf_at).
    """
    path = [0]
    cur = 0
    while True:
        p, _, _ = softmax64(np.asarray(target[cur], dtype=np.float64) / temperature)
        kids = children_of(parent, cur)
        r = p
        accepted = None
        if kids:
            q, _, _ = softmax64(np.asarray(draft[cur], dtype=np.float64) / temperature)
            for x in kids:
                t = token[x]
                a = min(1.0, r[t] / q[t]) if q[t] > 0 else 1.0
                if trace is not None:
                    trace.append(("accept", x, float(u_accept[x]), float(a)))
                if u_accept[x] < a:
                    accepted = x
                    break
                r = np.maximum(r - q, 0.0)
                z = r.sum()
                if z <= 0.0:            # p == q exactly: nothing left to sample, keep p
                    r = p
                    break
                r = r / z
        if accepted is None:
            cdf = np.cumsum(r)
            hit = np.nonzero(cdf > u_final)[0]
            bonus = int(hit[0]) if len(hit) else int(np.nonzero(r > 0)[0][-1])
            if trace is not None:
                trace.append(("final", float(u_final), float(cdf[bonus - 1]) if bonus else 0.0,
                              float(cdf[bonus])))
            return path, bonus
        cur = accepted
        path.append(cur)


def deterministic(parent, token, target, temperature, u_accept, u_final, trace=None):
    """Multi-candidate acceptance when every candidate is a deterministic proposal.

    At node cur with p = softmax(target[cur] / T) and r = p: children are tried in index order;
    the proposal distribution of child x is q = the point mass on tok = token[x], so x is accepted
    iff u_accept[x] < min(1, r[tok] / q[tok]) = r[tok]; otherwise r <- normalise(max(r - q, 0)),
    which removes tok from r.  After the last rejection (or at a leaf) the bonus token is the
    smallest j with cumsum(r)[j] > u_final.  ``trace`` as in `rejection`.
    """
    path = [0]
    cur = 0
    while True:
        p, _, _ = softmax64(np.asarray(target[cur], dtype=np.float64) / temperature)
        r = p
        accepted = None
        for x in children_of(parent, cur):
            t = token[x]
            q = np.zeros_like(p)
            q[t] = 1.0
            a = min(1.0, r[t] / q[t])
            if trace is not None:
                trace.append(("accept", x, float(u_accept[x]), float(a)))
            if u_accept[x] < a:
                accepted = x
                break
            r = np.maximum(r - q, 0.0)
            z = r.sum()
            if z <= 0.0:                # the whole mass sat on rejected tokens: keep p
                r = p
                break
            r = r / z
        if accepted is None:
            cdf = np.cumsum(r)
            hit = np.nonzero(cdf > u_final)[0]
            bonus = int(hit[0]) if len(hit) else int(np.nonzero(r > 0)[0][-1])
            if trace is not None:
                trace.append(("final", float(u_final), float(cdf[bonus - 1]) if bonus else 0.0,
                              float(cdf[bonus])))
            return path, bonus
        cur = accepted
        path.append(cur)
