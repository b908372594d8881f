"""Pins of the oracle's acceptance: brute force over all tree paths (greedy), the textbook chain
rule, degenerate uniforms / equal distributions, losslessness by chi-square, and the scalar
recurrence for the k-th residual against explicit residual vectors."""
import math

import numpy as np
import pytest
import scipy.stats

from oracle import accept
from oracle.row_stats import softmax64


def random_tree(rng, n, max_children=3):
    parent, nch = [-1], [0]
    for i in range(1, n):
        ok = [u for u in range(i) if nch[u] < max_children]
        p = ok[rng.integers(len(ok))]
        parent.append(p); nch.append(0); nch[p] += 1
    return np.array(parent)


@pytest.mark.parametrize("seed", range(10))
def test_greedy_brute_force(seed):
    rng = np.random.default_rng(seed)
    n, V = 12, 6
    parent = random_tree(rng, n)
    token = np.zeros(n, dtype=np.int64)
    for p in range(n):                                   # distinct tokens among siblings
        kids = [i for i in range(n) if parent[i] == p]
        token[kids] = rng.permutation(V)[: len(kids)]
    target = rng.integers(0, 4, (n, V)).astype(np.float64)        # many exact ties
    path, bonus = accept.greedy(parent, token, target)
    # brute force: a node is valid iff every token on its root path equals the first maximum of
    # the row before it; the accepted path is the deepest valid node's path
    first_max = [int(np.argmax(target[i])) for i in range(n)]      # np.argmax returns the first
    valid = [True] + [False] * (n - 1)
    for i in range(1, n):
        valid[i] = valid[parent[i]] and token[i] == first_max[parent[i]]
    depth = [0] * n
    for i in range(1, n):
        depth[i] = depth[parent[i]] + 1
    deepest = max((i for i in range(n) if valid[i]), key=lambda i: depth[i])
    want = []
    j = deepest
    while j != -1:
        want.append(j); j = parent[j]
    assert path == want[::-1]
    assert bonus == first_max[deepest]
    assert path[0] == 0 and all(parent[b] == a for a, b in zip(path, path[1:]))


def test_chain_is_textbook_speculative_sampling():
    rng = np.random.default_rng(3)
    n, V = 5, 7
    parent = np.arange(-1, n - 1)
    token = rng.integers(0, V, n)
    target, draft = rng.standard_normal((n, V)), rng.standard_normal((n, V))
    u = rng.random(n)
    path, bonus = accept.rejection(parent, token, target, draft, 1.0, u, 0.4)
    # textbook: accept token i+1 while u < min(1, p/q); at the first rejection sample from
    # normalise(max(p - q, 0)); if all accepted sample from p of the last node
    cur, want = 0, [0]
    while cur + 1 < n:
        p = np.exp(target[cur]) / np.exp(target[cur]).sum()
        q = np.exp(draft[cur]) / np.exp(draft[cur]).sum()
        t = token[cur + 1]
        if u[cur + 1] < min(1.0, p[t] / q[t]):
            cur += 1; want.append(cur)
            continue
        res = np.maximum(p - q, 0); res /= res.sum()
        break
    else:
        res = np.exp(target[cur]) / np.exp(target[cur]).sum()
    assert path == want
    assert bonus == int(np.searchsorted(np.cumsum(res), 0.4, side="right"))


def test_degenerate_uniforms_and_equal_distributions():
    rng = np.random.default_rng(4)
    n, V = 9, 11
    parent = np.array([-1, 0, 0, 1, 1, 3, 3, 5, 5])
    token = rng.integers(0, V, n)
    target, draft = rng.standard_normal((n, V)), rng.standard_normal((n, V))
    path, _ = accept.rejection(parent, token, target, draft, 1.0, np.zeros(n), 0.5)
    assert path == [0, 1, 3, 5, 7]                        # u = 0: first child always accepted
    path, _ = accept.rejection(parent, token, target, target, 0.7, np.full(n, 0.999999), 0.5)
    assert path == [0, 1, 3, 5, 7]                        # p == q: acceptance probability is 1
    path, bonus = accept.rejection(parent, token, target, draft, 1.0, np.full(n, 2.0), 0.0)
    assert path == [0]                                    # u > 1 rejects every candidate
    p = softmax64(target[0])[0]; q = softmax64(draft[0])[0]
    r = p
    for _ in range(2):
        r = np.maximum(r - q, 0); r /= r.sum()
    assert bonus == int(np.nonzero(r > 0)[0][0])          # u_final = 0 -> first token with mass


def test_temperature_scales_both_models():
    rng = np.random.default_rng(5)
    parent = np.array([-1, 0]); token = np.array([0, 3])
    target, draft = rng.standard_normal((2, 6)), rng.standard_normal((2, 6))
    T = 0.5
    p = softmax64(target[0] / T)[0]; q = softmax64(draft[0] / T)[0]
    a = min(1.0, p[3] / q[3])
    lo, _ = accept.rejection(parent, token, target, draft, T, np.array([0, a * 0.999]), 0.5)
    hi, _ = accept.rejection(parent, token, target, draft, T, np.array([0, min(a * 1.001, 1.0)]), 0.5)
    assert lo == [0, 1] and (hi == [0] or a == 1.0)


def test_lossless_output_distribution():
    """One tree level whose k candidate tokens are drawn i.i.d. from the draft distribution:
    the token emitted after the root must follow the target distribution exactly."""
    rng = np.random.default_rng(6)
    V, k, trials = 8, 3, 40000
    target = rng.standard_normal((k + 1, V)) * 1.5
    draft = rng.standard_normal((k + 1, V)) * 1.5
    p = softmax64(target[0])[0]; q = softmax64(draft[0])[0]
    parent = np.array([-1] + [0] * k)
    counts = np.zeros(V)
    for _ in range(trials):
        token = np.concatenate([[0], rng.choice(V, size=k, p=q)])
        path, bonus = accept.rejection(parent, token, target, draft, 1.0, rng.random(k + 1), rng.random())
        counts[token[path[1]] if len(path) > 1 else bonus] += 1
    chi2 = ((counts - trials * p) ** 2 / (trials * p)).sum()
    assert scipy.stats.chi2.sf(chi2, V - 1) > 1e-3


def test_residual_scalar_recurrence():
    """After k rejections the residual equals max(p - c_k q, 0) / W_k with c_0 = 0, W_0 = 1,
    c_(k+1) = c_k + W_k, W_k = sum max(p - c_k q, 0): checked against explicit residual vectors
    recovered from the accept-test probabilities the oracle reports."""
    rng = np.random.default_rng(7)
    V, k = 50, 6
    target, draft = rng.standard_normal((k + 1, V)) * 2, rng.standard_normal((k + 1, V))
    p = softmax64(target[0])[0]; q = softmax64(draft[0])[0]
    parent = np.array([-1] + [0] * k)
    token = np.concatenate([[0], rng.permutation(V)[:k]])
    trace = []
    accept.rejection(parent, token, target, draft, 1.0, np.full(k + 1, 2.0), 0.3, trace=trace)
    r, c, W = p.copy(), 0.0, 1.0
    for j, (_, x, _, a) in enumerate(t for t in trace if t[0] == "accept"):
        t = token[x]
        assert a == pytest.approx(min(1.0, r[t] / q[t]), rel=1e-12)
        assert np.allclose(r, np.maximum(p - c * q, 0) / W, atol=1e-14)
        r = np.maximum(r - q, 0); r /= r.sum()
        c = c + W
        W = np.maximum(p - c * q, 0).sum()
    final = [t for t in trace if t[0] == "final"][0]
    cdf = np.cumsum(np.maximum(p - c * q, 0) / W)
    j = int(np.searchsorted(cdf, 0.3, side="right"))
    assert final[3] == pytest.approx(cdf[j], rel=1e-12)


# ---- deterministic proposals (q = point mass on the candidate's token) ------------------------------------

def test_deterministic_chain_equals_rejection_with_point_mass_draft():
    """On a chain every node has one candidate, and a draft row that puts all its mass on that candidate's token
    turns the general sampler (pinned above) into the deterministic-proposal one."""
    rng = np.random.default_rng(11)
    n, V = 6, 9
    parent = np.arange(-1, n - 1)
    for trial in range(200):
        token = rng.integers(0, V, n)
        target = rng.standard_normal((n, V)) * 2.0
        draft = np.full((n, V), -1e30)
        for i in range(n - 1):
            draft[i, token[i + 1]] = 0.0            # softmax: the point mass on the child's token
        draft[n - 1, 0] = 0.0
        u, uf = rng.random(n), rng.random()
        assert accept.deterministic(parent, token, target, 0.8, u, uf) == \
            accept.rejection(parent, token, target, draft, 0.8, u, uf)


def test_deterministic_closed_form_of_sibling_tests():
    """The k-th sibling is accepted with probability p(t_k) / (1 - sum of p over the tokens rejected before it);
    the bonus token comes from p with the rejected tokens removed."""
    rng = np.random.default_rng(12)
    V, k = 10, 4
    parent = np.array([-1] + [0] * k)
    for trial in range(200):
        target = rng.standard_normal((k + 1, V)) * 1.5
        p = softmax64(target[0])[0]
        token = np.concatenate([[0], rng.choice(V, size=k, replace=False)])
        u, uf = rng.random(k + 1), rng.random()
        trace = []
        path, bonus = accept.deterministic(parent, token, target, 1.0, u, uf, trace=trace)
        gone, want = 0.0, None
        for x in range(1, k + 1):
            a = p[token[x]] / (1.0 - gone)
            if u[x] < min(1.0, a):
                want = x
                break
            gone += p[token[x]]
        if want is not None:
            assert path == [0, want]
        else:
            r = p.copy(); r[token[1:]] = 0.0; r /= r.sum()
            assert path == [0] and bonus == int(np.searchsorted(np.cumsum(r), uf, side="right"))
    # u = 0 accepts the first candidate whose token has any mass
    path, _ = accept.deterministic(parent, token, target, 1.0, np.zeros(k + 1), 0.5)
    assert path == [0, 1]


def test_deterministic_lossless_output_distribution():
    """Whatever fixed tokens the candidates carry, the token emitted after the root follows the target distribution."""
    rng = np.random.default_rng(13)
    V, k, trials = 8, 3, 40000
    target = rng.standard_normal((k + 1, V)) * 1.5
    p = softmax64(target[0])[0]
    parent = np.array([-1] + [0] * k)
    token = np.array([0, 5, 2, 7])                  # fixed proposals (e.g. the draft model's top-3)
    counts = np.zeros(V)
    for _ in range(trials):
        path, bonus = accept.deterministic(parent, token, target, 1.0, rng.random(k + 1), rng.random())
        counts[token[path[1]] if len(path) > 1 else bonus] += 1
    chi2 = ((counts - trials * p) ** 2 / (trials * p)).sum()
    assert scipy.stats.chi2.sf(chi2, V - 1) > 1e-3
