"""Oracle: draft-tree expansion and reranking (test infrastructure only).

Sec. 2.2 of the paper (the EAGLE-2 scheme HeteroSpec builds on): the draft tree grows level by
level.  At each level the draft model is run on a frontier of at most k nodes; every frontier node
gets the k most likely next tokens as children, the value of a node is the product of the
confidences along its path, V_i = prod c_j (kept in log form, S = ln V), and the k children with the
largest value form the next frontier.  After the last level all candidates are reranked: the N with
the largest value (root included) are the tree that goes to verification; because a child's value
never exceeds its parent's, that set is closed under ancestors.  Sec. 4.3 (dynamic extended
drafting) only changes how many levels are grown (d' = d_base + Delta) and how many nodes survive
the reranking (N' instead of N); both are arguments here.

Plain python lists, float64; ties go to the candidate created first (lower candidate id).
"""

import numpy as np

from .row_stats import softmax64, topk_indices


def expand(draft_row, depth, k):
    """Grows the candidate tree to `depth` levels.

    draft_row(cand_id, path_tokens) -> the draft model's logits after that candidate (a 1-D array);
    it is only called for frontier nodes.  Returns dict(parent, token, depth, logc, S, frontiers)
    with candidates in creation order (candidate 0 is the root, parents precede children) and
    frontiers[l] = the candidate ids expanded at level l + 1.
    """
    parent, token, dep, logc, S = [-1], [-1], [0], [0.0], [0.0]
    paths = [[]]
    frontier = [0]
    frontiers = []
    for level in range(1, depth + 1):
        frontiers.append(list(frontier))
        new = []
        for f in frontier:
            row = np.asarray(draft_row(f, paths[f]), dtype=np.float64)
            _, _, lse = softmax64(row)
            for t in topk_indices(row, k):
                parent.append(f); token.append(int(t)); dep.append(level)
                lc = float(row[t] - lse)
                logc.append(lc); S.append(S[f] + lc)
                paths.append(paths[f] + [int(t)])
                new.append(len(parent) - 1)
        frontier = sorted(new, key=lambda c: (-S[c], c))[:k]
    return dict(parent=np.array(parent), token=np.array(token), depth=np.array(dep),
                logc=np.array(logc), S=np.array(S), frontiers=frontiers)


def rerank(cand, n_top):
    """The n_top candidates with the largest value (S descending, candidate id ascending), as a
    tree in creation order: returns dict(cand_id, parent, token, depth) with parent re-indexed to
    the kept nodes.  The root (value 1) is always among them."""
    S = cand["S"]
    order = sorted(range(len(S)), key=lambda c: (-S[c], c))[: min(n_top, len(S))]
    keep = sorted(order)
    new_index = {c: i for i, c in enumerate(keep)}
    par = [-1 if cand["parent"][c] < 0 else new_index[int(cand["parent"][c])] for c in keep]   # KeyError = not closed
    return dict(cand_id=np.array(keep), parent=np.array(par), token=cand["token"][keep],
                depth=cand["depth"][keep])
