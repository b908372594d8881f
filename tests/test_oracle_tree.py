"""Pins of the oracle's path aggregation, stratification, pruning and mask: Eq. 1 on chains,
brute-force path enumeration, the hand-evaluated policy table, subset brute force, closure."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import tree

GOLD = os.path.join(os.path.dirname(__file__), "golden", "policy_table.txt")


def policy(th=(1, 2, 3, 4, 5, 6, 7), d_base=8, alpha=4, n_default=60, k=3, **kw):
    p = dict(thresholds=list(th), d_base=d_base, alpha=alpha, n_default=n_default, top_k=k,
             gamma_pct=[30, 60, 100], phi_mode=0, pstar_mode=0, entropy_mode=0)
    p.update(kw)
    return p


def random_tree(rng, n, max_depth=6, max_children=4):
    parent, depth, nch = [-1], [0], [0]
    for i in range(1, n):
        ok = [u for u in range(i) if depth[u] < max_depth and nch[u] < max_children]
        p = ok[rng.integers(len(ok))]
        parent.append(p); depth.append(depth[p] + 1); nch.append(0); nch[p] += 1
    return np.array(parent)


def entropy_of_topk(row, k):
    """Eq. 1 inner sum written out independently: sort probabilities, renormalise, -sum p ln p."""
    e = [math.exp(x - max(row)) for x in row]
    p = sorted((x / sum(e) for x in e), reverse=True)[:k]
    z = sum(p)
    return -sum((x / z) * math.log(x / z) for x in p if x > 0)


def test_chain_is_eq1():
    rng = np.random.default_rng(0)
    n, V, K = 7, 50, 3
    logits = rng.standard_normal((n, V)) * 2
    parent = np.arange(-1, n - 1)
    token = rng.integers(0, V, n)
    sc = tree.tree_scores(parent, token, logits, policy(k=K, d_base=6))
    phi = 0.0
    s = 0.0
    for t in range(1, n):
        phi += entropy_of_topk(list(logits[t - 1]), K)
        row = logits[t - 1]
        s += row[token[t]] - math.log(sum(math.exp(x) for x in row))
        assert sc["Phi"][t] == pytest.approx(phi, rel=1e-12)
        assert sc["S"][t] == pytest.approx(s, rel=1e-12)
    assert sc["pstar_node"] == 6 and sc["phi_star"] == pytest.approx(phi, rel=1e-12)
    inc = tree.tree_scores(parent, token, logits, policy(k=K, d_base=6, phi_mode=1))
    assert inc["phi_star"] == pytest.approx(phi + entropy_of_topk(list(logits[6]), K), rel=1e-12)


@pytest.mark.parametrize("seed", range(6))
def test_brute_force_paths(seed):
    rng = np.random.default_rng(seed)
    n, V, K = 12, 40, 4
    parent = random_tree(rng, n, max_depth=4)
    token = rng.integers(0, V, n)
    logits = rng.standard_normal((n, V)) * rng.uniform(0.3, 3, (n, 1))
    d_base = 3
    sc = tree.tree_scores(parent, token, logits, policy(k=K, d_base=d_base))
    # enumerate every root->node path explicitly
    paths = {}
    for i in range(n):
        p, j = [], i
        while j != -1:
            p.append(j); j = parent[j]
        paths[i] = p[::-1]
    lp = lambda r, t: logits[r][t] - math.log(sum(math.exp(x) for x in logits[r]))
    for i, p in paths.items():
        phi = sum(entropy_of_topk(list(logits[a]), K) for a in p[:-1])
        s = sum(lp(a, token[b]) for a, b in zip(p[:-1], p[1:]))
        assert sc["Phi"][i] == pytest.approx(phi, rel=1e-11, abs=1e-12)
        assert sc["S"][i] == pytest.approx(s, rel=1e-11, abs=1e-12)
        assert sc["depth"][i] == len(p) - 1
        assert sc["S"][i] <= (sc["S"][parent[i]] if i else 0.0) + 1e-15    # V_i bounded by ancestors
    t_eval = min(d_base, max(len(p) - 1 for p in paths.values()))
    full = [i for i, p in paths.items() if len(p) - 1 == t_eval]
    best = max(full, key=lambda i: (lp(parent[i], token[i]), -i))
    assert sc["pstar_node"] == best
    cum = tree.tree_scores(parent, token, logits, policy(k=K, d_base=d_base, pstar_mode=1))
    assert cum["pstar_node"] == max(full, key=lambda i: (cum["S"][i], -i))


def test_policy_table_golden():
    rows = [list(map(int, l.split())) for l in open(GOLD) if l.strip() and not l.startswith("#")]
    assert len(rows) >= 9
    th = [1, 2, 3, 4, 5, 6, 7]
    for n_default, d_base, alpha, b, d_prime, n_prime in rows:
        pol = policy(th, d_base=d_base, alpha=alpha, n_default=n_default)
        phi = 0.5 if b == 0 else th[b - 1] + 0.5
        assert tree.stratify(phi, pol) == (b, d_prime, n_prime)


def test_bin_boundaries():
    pol = policy([1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 7.0])
    assert tree.stratify(0.999, pol)[0] == 0
    assert tree.stratify(1.0, pol)[0] == 1          # bin = number of thresholds <= phi
    assert tree.stratify(6.999, pol)[0] == 6
    assert tree.stratify(1e9, pol)[0] == 7


def closed(keep, parent):
    return all(parent[i] < 0 or parent[i] in keep for i in keep)


@pytest.mark.parametrize("seed", range(8))
def test_prune_subset_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    n = 10
    parent = random_tree(rng, n, max_depth=4, max_children=3)
    d = tree.depths(parent)
    S = np.zeros(n)
    for i in range(1, n):
        S[i] = S[parent[i]] - rng.uniform(0.05, 2.0)
    for d_prime, n_prime in ((2, 4), (4, 6), (9, 7), (9, 50), (1, 3)):
        out = tree.prune(parent, S, d_prime, n_prime)
        keep = set(out["keep_idx"].tolist())
        elig = [i for i in range(n) if d[i] <= d_prime]
        size = min(n_prime, len(elig))
        assert len(keep) == size and 0 in keep and closed(keep, parent)
        best, best_sets = -1e300, []
        for sub in itertools.combinations(elig, size):
            ss = set(sub)
            if 0 in ss and closed(ss, parent):
                tot = sum(S[i] for i in sub)
                if tot > best + 1e-12:
                    best, best_sets = tot, [ss]
                elif abs(tot - best) <= 1e-12:
                    best_sets.append(ss)
        assert best_sets == [keep]
        dropped = [i for i in elig if i not in keep]
        if dropped:
            assert max(S[i] for i in dropped) <= min(S[i] for i in keep)


def test_prune_identity_and_ties():
    parent = np.array([-1, 0, 0, 1, 1, 2])
    S = np.array([0.0, -1.0, -1.0, -1.0, -2.0, -1.0])        # exact ties, also child == parent
    out = tree.prune(parent, S, 10, 99)
    assert out["keep_idx"].tolist() == list(range(6))
    assert out["new_parent"].tolist() == parent.tolist()
    out = tree.prune(parent, S, 10, 4)                       # ties break to the lowest index
    assert out["keep_idx"].tolist() == [0, 1, 2, 3]
    assert out["rank"].tolist() == [0, 1, 2, 3]
    out = tree.prune(parent, S, 1, 99)                       # depth cap
    assert out["keep_idx"].tolist() == [0, 1, 2]


@pytest.mark.parametrize("seed", range(4))
def test_mask_is_transitive_closure(seed):
    rng = np.random.default_rng(seed)
    n = 20
    parent = random_tree(rng, n)
    S = np.zeros(n)
    for i in range(1, n):
        S[i] = S[parent[i]] - rng.uniform(0.1, 1.0)
    out = tree.prune(parent, S, 5, 13)
    m = len(out["keep_idx"])
    A = np.eye(m, dtype=np.int64)
    for i in range(m):
        if out["new_parent"][i] >= 0:
            A[i, out["new_parent"][i]] = 1
    R = A.copy()
    for _ in range(m):
        R = ((R @ A) > 0).astype(np.int64)
    assert np.array_equal(R.astype(bool), out["mask"])
    assert np.array_equal(out["mask"].sum(1), out["new_depth"] + 1)
    assert not np.triu(out["mask"], 1).any()
    # compacted parents point at the same original nodes
    for new, old in enumerate(out["keep_idx"]):
        if parent[old] >= 0:
            assert out["keep_idx"][out["new_parent"][new]] == parent[old]
