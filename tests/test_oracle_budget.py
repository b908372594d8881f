"""Pins of the budget-reallocation oracle (App. A.8): the budget is respected, nobody drops below the root or rises
above its eligible nodes, the order of service follows the SLO classes, and on tiny batches the result equals the
lexicographically best allocation found by brute force."""
import itertools

import numpy as np
import pytest

from oracle import budget


def brute_force(n_prime, eligible, slo, T):
    """All allocations with 1 <= n_b <= max(eligible_b, 1) and sum <= max(T, B); the winner serves the sequences
    in SLO order: under budget nobody gets less than its request and, going down the order, each gets as much as
    possible; over budget nobody gets more than its request and, going down the order, each keeps as much as possible."""
    B = len(n_prime)
    base = [max(1, min(n_prime[b], eligible[b])) for b in range(B)]
    order = sorted(range(B), key=lambda b: (slo[b], b))
    cap = max(T, B)
    best = None
    for alloc in itertools.product(*[range(1, max(eligible[b], 1) + 1) for b in range(B)]):
        if sum(alloc) > cap:
            continue
        if sum(base) <= T:
            if any(alloc[b] < base[b] for b in range(B)):
                continue
        else:
            if any(alloc[b] > base[b] for b in range(B)):
                continue
        key = tuple(alloc[b] for b in order)
        if best is None or key > best[0]:
            best = (key, alloc)
    return list(best[1])


@pytest.mark.parametrize("seed", range(40))
def test_equals_brute_force_on_tiny_batches(seed):
    rng = np.random.default_rng(seed)
    B = int(rng.integers(1, 5))
    eligible = [int(v) for v in rng.integers(1, 7, B)]
    n_prime = [int(v) for v in rng.integers(1, 8, B)]
    slo = [int(v) for v in rng.integers(0, 3, B)]
    T = int(rng.integers(1, 20))
    assert budget.reallocate(n_prime, eligible, slo, T) == brute_force(n_prime, eligible, slo, T)


def test_properties_on_larger_batches():
    rng = np.random.default_rng(1)
    for _ in range(200):
        B = int(rng.integers(1, 40))
        eligible = rng.integers(1, 97, B).tolist()
        n_prime = rng.choice([22, 39, 62, 60], B).tolist()
        slo = rng.integers(0, 4, B).tolist()
        T = int(rng.integers(B, 60 * B))
        out = budget.reallocate(n_prime, eligible, slo, T)
        base = [max(1, min(n_prime[b], eligible[b])) for b in range(B)]
        assert all(1 <= out[b] <= max(eligible[b], 1) for b in range(B))
        assert sum(out) <= max(T, B)
        if sum(base) <= T:
            assert all(out[b] >= base[b] for b in range(B))
            # nothing is left over while somebody could still take more
            assert sum(out) == min(T, sum(max(e, 1) for e in eligible))
            # a stricter class is never left short while a looser one got extra
            for a in range(B):
                for c in range(B):
                    if (slo[a], a) < (slo[c], c) and out[c] > base[c]:
                        assert out[a] == max(eligible[a], 1)
        else:
            assert all(out[b] <= base[b] for b in range(B))
            assert sum(out) == max(T, B) or all(o == 1 for o in out)


def test_worked_example():
    # three requests of the policy sizes 22 / 39 / 60 on trees of 60 eligible nodes, budget 128: 7 tokens are left
    # over and go to the strictest class (sequence 1), then nothing remains
    assert budget.reallocate([22, 39, 60], [60, 60, 60], [1, 0, 2], 128) == [22, 46, 60]
    # budget 100: 21 tokens must come back, from the loosest class first
    assert budget.reallocate([22, 39, 60], [60, 60, 60], [1, 0, 2], 100) == [22, 39, 39]
    # budget below one token per sequence: everybody keeps the root
    assert budget.reallocate([22, 39, 60], [60, 60, 60], [1, 0, 2], 2) == [1, 1, 1]
