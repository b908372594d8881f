"""Pins of the expansion / reranking oracle (Sec. 2.2): brute force over the complete k-ary tree on tiny
cases, monotone values, ancestor closure, and reranking = Top-N pruning of the full candidate tree."""
import itertools

import numpy as np
import pytest

from oracle import expand as oexp
from oracle import tree as otree


def make_model(vocab, seed):
    """A deterministic toy draft model: the row after a token path depends only on the path."""
    def row(path):
        r = np.random.default_rng([seed, len(path)] + list(path))
        return r.standard_normal(vocab) * 2.0
    return row


@pytest.mark.parametrize("seed", range(4))
def test_frontier_and_values_match_brute_force(seed):
    vocab, k, depth = 7, 2, 3
    model = make_model(vocab, seed)
    cand = oexp.expand(lambda c, path: model(path), depth, k)
    # brute force: the full k-ary tree of top-k tokens, level by level, keeping the k best paths per level
    logp = lambda path: model(path) - np.log(np.exp(model(path)).sum())
    frontier = [()]
    seen = {(): 0.0}
    for level in range(depth):
        new = {}
        for path in frontier:
            lp = logp(list(path))
            best = sorted(range(vocab), key=lambda t: (-lp[t], t))[:k]
            for t in best:
                new[path + (t,)] = seen[path] + lp[t]
        seen.update(new)
        frontier = sorted(new, key=lambda q: -new[q])[:k]          # (no ties in these draws)
    assert len(cand["S"]) == len(seen)
    got = {}
    for c in range(len(cand["S"])):
        path, a = [], c
        while cand["parent"][a] >= 0:
            path.append(int(cand["token"][a])); a = int(cand["parent"][a])
        got[tuple(reversed(path))] = cand["S"][c]
    assert set(got) == set(seen)
    for q in seen:
        assert abs(got[q] - seen[q]) < 1e-12
    # number of candidates: 1 + k + (depth - 1) k^2
    assert len(seen) == 1 + k + (depth - 1) * k * k


@pytest.mark.parametrize("seed", range(4))
def test_values_never_grow_along_a_path_and_rerank_is_closed(seed):
    vocab, k, depth = 50, 4, 5
    model = make_model(vocab, 100 + seed)
    cand = oexp.expand(lambda c, path: model(path), depth, k)
    S, par = cand["S"], cand["parent"]
    assert all(S[c] <= S[par[c]] + 1e-15 for c in range(1, len(S)))
    assert all(par[c] < c for c in range(1, len(S)))
    for n_top in (1, 5, 17, len(S), len(S) + 3):
        t = oexp.rerank(cand, n_top)
        assert t["cand_id"][0] == 0 and len(t["cand_id"]) == min(n_top, len(S))
        kept = set(int(c) for c in t["cand_id"])
        assert all(int(par[c]) in kept for c in kept if c != 0)
        # the kept set is what Top-N pruning of the full candidate tree keeps (same key, same tie-break)
        pr = otree.prune(par, S, depth, n_top)
        assert np.array_equal(pr["keep_idx"], t["cand_id"]) and np.array_equal(pr["new_parent"], t["parent"])


def test_ties_go_to_the_candidate_created_first():
    # a model whose rows are constant: every token ties, children are tokens 0..k-1, every path has the same value per level
    cand = oexp.expand(lambda c, path: np.zeros(6), 3, 2)
    assert cand["token"].tolist() == [-1, 0, 1, 0, 1, 0, 1, 0, 1, 0, 1]
    assert cand["frontiers"] == [[0], [1, 2], [3, 4]]
    t = oexp.rerank(cand, 4)
    assert t["cand_id"].tolist() == [0, 1, 2, 3]
