"""Oracle: token-budget reallocation across the sequences of a batch (test infrastructure only).

App. A.8 of the paper ("More Discussion"): serving systems cap the tokens one forward pass of the
target model may process (the hardware budget); Top-N pruning makes low-entropy requests need less of
it "without sacrificing acceptance rates", which "enables budget reallocation to stricter SLO
requests".  The paper gives no algorithm; the reading implemented here is the simplest one that has
these properties:

  * every sequence b first asks for what the policy gives it, base_b = min(N'_b, eligible_b), where
    eligible_b is the number of drafted nodes within its depth limit d'_b (at least 1: the root);
  * if the requests fit the budget T, the tokens left over, T - sum(base), go to the sequences in
    order of SLO class (smaller class = stricter, served first; ties: lower sequence index), each
    taking as many more of its eligible nodes as are left;
  * if they do not fit, the excess is taken back in the opposite order (loosest class first, ties:
    higher index), never below one node (the root) per sequence.

The result n_final_b replaces N'_b in the Top-N reranking, so every tree stays closed under
ancestors; the sum is at most max(T, B).
"""


def reallocate(n_prime, eligible, slo_class, budget):
    """n_prime, eligible, slo_class: per-sequence lists; budget: tokens per forward pass.
    Returns the per-sequence node counts."""
    B = len(n_prime)
    base = [max(1, min(int(n_prime[b]), int(eligible[b]))) for b in range(B)]
    out = list(base)
    total = sum(base)
    if total <= budget:
        left = budget - total
        for b in sorted(range(B), key=lambda b: (slo_class[b], b)):
            extra = min(left, max(int(eligible[b]), 1) - base[b])
            if extra > 0:
                out[b] += extra
                left -= extra
    else:
        excess = total - budget
        for b in sorted(range(B), key=lambda b: (-slo_class[b], -b)):
            cut = min(excess, base[b] - 1)
            if cut > 0:
                out[b] -= cut
                excess -= cut
    return out
