"""Oracle steps 2-4: path aggregation, stratification, pruning, tree mask.

TEST INFRASTRUCTURE ONLY; float64, plain loops over tree nodes.

Conventions: nodes are in topological order (parent index < own index), node 0
is the root (the last accepted token, depth 0) and ``logits[n]`` is the draft
model's next-token distribution after node n, i.e. the distribution the tokens
of n's children were taken from.
"""

import numpy as np

from .row_stats import row_stats


def depths(parent):
    d = np.zeros(len(parent), dtype=np.int64)
    for n in range(1, len(parent)):
        d[n] = d[parent[n]] + 1
    return d


def tree_scores(parent, token, logits, policy, stats=None):
    """Cumulative meta-path Top-K entropy and path confidence of every node.

    logc[n]  = ln c_n, the draft log-probability of token[n] under the row of parent(n)
    S[n]     = sum of logc along root -> n  (= ln V_i of Sec. 2.2, V_i = prod c_j)
    Phi[n]   = Eq. 1 for the path root -> n: the sum over t = 1..T of the Top-K entropy of
               the distribution x_t was drawn from (the row of x_t's parent).  With
               policy["phi_mode"] == 1 the node's own row is added as well.
    P*       = the path ending in the node of depth T_eval = min(d_base, tree depth) whose
               final token has the highest confidence (Sec. 4.1): largest logc (pstar_mode 0)
               or largest S (pstar_mode 1); ties go to the lowest index.
    Returns dict(logc, S, Phi, depth, pstar_node, phi_star, I).
    """
    n = len(parent)
    K = policy["top_k"]
    if stats is None:
        stats = [row_stats(logits[i], K) for i in range(n)]
    I_key = "I_topk" if policy.get("entropy_mode", 0) == 0 else "I_trunc"
    I = np.array([s[I_key] for s in stats], dtype=np.float64)
    lse = np.array([s["lse"] for s in stats], dtype=np.float64)
    d = depths(parent)
    logc = np.zeros(n); S = np.zeros(n); Phi = np.zeros(n)
    for i in range(1, n):
        p = parent[i]
        logc[i] = float(logits[p][token[i]]) - lse[p]
        S[i] = S[p] + logc[i]
        Phi[i] = Phi[p] + I[p]
    Phi_out = Phi + I if policy.get("phi_mode", 0) == 1 else Phi
    t_eval = min(policy["d_base"], int(d.max()))
    key = logc if policy.get("pstar_mode", 0) == 0 else S
    cand = [i for i in range(n) if d[i] == t_eval]
    pstar = cand[0]
    for i in cand[1:]:
        if key[i] > key[pstar]:
            pstar = i
    return dict(logc=logc, S=S, Phi=Phi_out, depth=d, pstar_node=int(pstar),
                phi_star=float(Phi_out[pstar]), I=I)


def stratify(phi_star, policy):
    """Entropy bin and the (d', N') it selects (Sec. 4.2-4.3).

    bin = number of thresholds <= phi_star (eight bins B_0..B_7, ascending entropy).
    For the low-entropy bins i in {0, 1, 2}: Delta = alpha - i,
        d' = d_base + Delta,  N' = gamma_(i+1) * N_default + Delta,  gamma = 0.3, 0.6, 1.0
    (gamma * N rounded half-up); the other bins keep d_base and N_default.
    """
    th = policy["thresholds"]
    b = sum(1 for t in th if phi_star >= t)
    if b <= 2:
        delta = policy["alpha"] - b
        d_prime = policy["d_base"] + delta
        n_prime = (policy["gamma_pct"][b] * policy["n_default"] + 50) // 100 + delta
    else:
        d_prime, n_prime = policy["d_base"], policy["n_default"]
    return b, d_prime, n_prime


def prune(parent, S, d_prime, n_prime):
    """Top-N' reranking (Sec. 2.2 with N -> N'): among nodes of depth <= d', keep the N'
    with the largest path confidence S (ties: lowest index), compact them preserving order,
    re-index parents, and build the ancestor-or-self visibility mask.

    Returns dict(keep_idx, new_parent, new_depth, rank, mask) with mask[i, j] = True iff
    kept node j is kept node i itself or one of its ancestors.
    """
    n = len(parent)
    d = depths(parent)
    elig = [i for i in range(n) if d[i] <= d_prime]
    order = sorted(elig, key=lambda i: (-S[i], i))
    keep = sorted(order[: min(n_prime, len(order))])
    rank_of = {i: r for r, i in enumerate(order)}
    new_index = {old: new for new, old in enumerate(keep)}
    m = len(keep)
    new_parent = np.full(m, -1, dtype=np.int64)
    for new, old in enumerate(keep):
        if parent[old] >= 0:
            new_parent[new] = new_index[parent[old]]      # KeyError here = not ancestor-closed
    mask = np.zeros((m, m), dtype=bool)
    for i in range(m):
        j = i
        while j >= 0:
            mask[i, j] = True
            j = new_parent[j]
    return dict(keep_idx=np.array(keep, dtype=np.int64), new_parent=new_parent,
                new_depth=d[keep], rank=np.array([rank_of[i] for i in keep], dtype=np.int64),
                mask=mask)


def margins(scores, policy, n_primes=None):
    """Distances of the float decisions from their boundaries, for guard-banding test inputs:
    phi_star to the nearest threshold; for every N' of the policy the gap between the
    confidence of rank N'-1 and rank N'; the P* key gap to the runner-up."""
    th = np.asarray(policy["thresholds"], dtype=np.float64)
    m_bin = float(np.min(np.abs(th - scores["phi_star"]))) if len(th) else np.inf
    S, d = scores["S"], scores["depth"]
    if n_primes is None:
        n_primes = sorted({stratify(x, policy)[2] for x in (-np.inf, *th)})
    m_rank = np.inf
    for b in range(len(th) + 1):
        _, dp, npr = stratify(-np.inf if b == 0 else th[b - 1], policy)
        elig = sorted((i for i in range(len(S)) if d[i] <= dp), key=lambda i: (-S[i], i))
        if 0 < npr < len(elig):
            m_rank = min(m_rank, S[elig[npr - 1]] - S[elig[npr]])
    key = scores["logc"] if policy.get("pstar_mode", 0) == 0 else S
    t_eval = d[scores["pstar_node"]]
    others = [key[i] for i in range(len(S)) if d[i] == t_eval and i != scores["pstar_node"]]
    m_pstar = float(key[scores["pstar_node"]] - max(others)) if others else np.inf
    return dict(bin=m_bin, rank=float(m_rank), pstar=m_pstar)
