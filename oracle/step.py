"""Oracle: one whole verification step over a ragged batch (test infrastructure only).

Chains the per-step oracles in the order of the decode loop (Sec. 4: quantify -> stratify ->
prune -> verify with tree attention -> accept) on a batch laid out as the input generators
emit it.  Plain per-sequence loops; used by the parity tests, the smoke check and the
benchmark's CPU-baseline timing.
"""

import numpy as np

from . import accept, attention, philox, row_stats, tree


def _widen(x):
    x = np.asarray(x)
    if x.dtype == np.uint16:                       # bfloat16 bit patterns
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return x.astype(np.float64)


def quantify(batch, policy, b):
    lo, hi = batch["node_off"][b], batch["node_off"][b + 1]
    logits = _widen(batch["draft"][lo:hi])
    stats = [row_stats.row_stats(r, policy["top_k"]) for r in logits]
    sc = tree.tree_scores(batch["parent"][lo:hi], batch["token"][lo:hi], logits, policy, stats=stats)
    return stats, sc


def stratify_prune(batch, policy, b, sc):
    lo, hi = batch["node_off"][b], batch["node_off"][b + 1]
    bin_, d_prime, n_prime = tree.stratify(sc["phi_star"], policy)
    pr = tree.prune(batch["parent"][lo:hi], sc["S"], d_prime, n_prime)
    pr.update(bin=bin_, d_prime=d_prime, n_prime=n_prime)
    return pr


def verify_attention(batch, b, pr, rows=None):
    cfg = batch["cfg"]
    lo = batch["node_off"][b]
    k0, k1 = batch["kv_off"][b], batch["kv_off"][b + 1]
    keep = lo + pr["keep_idx"]
    return attention.tree_attention(_widen(batch["q"][keep]), _widen(batch["k_tree"][keep]),
                                    _widen(batch["v_tree"][keep]), _widen(batch["k_cache"][k0:k1]),
                                    _widen(batch["v_cache"][k0:k1]), pr["mask"],
                                    cfg.head_dim ** -0.5, rows=rows)


def accept_path(batch, b, pr, trace=None):
    lo = batch["node_off"][b]
    keep = lo + pr["keep_idx"]
    token = batch["token"][keep]
    target = _widen(batch["target"][keep])
    if batch["mode"][b] == 0:
        path, bonus = accept.greedy(pr["new_parent"], token, target)
    elif batch["mode"][b] == 2:
        seed, off = batch["philox_seed"], batch["philox_offset"]
        u_acc = np.array([philox.uniform(seed, off, b, int(orig), 0) for orig in pr["keep_idx"]])
        u_fin = philox.uniform(seed, off, b, 0, 1)
        path, bonus = accept.deterministic(pr["new_parent"], token, target, float(batch["temperature"][b]),
                                           u_acc, u_fin, trace=trace)
    else:
        draft = _widen(batch["draft"][keep])
        seed, off = batch["philox_seed"], batch["philox_offset"]
        u_acc = np.array([philox.uniform(seed, off, b, int(orig), 0) for orig in pr["keep_idx"]])
        u_fin = philox.uniform(seed, off, b, 0, 1)
        path, bonus = accept.rejection(pr["new_parent"], token, target, draft,
                                       float(batch["temperature"][b]), u_acc, u_fin, trace=trace)
    return dict(path_compact=path, path_nodes=[int(pr["keep_idx"][i]) for i in path],
                path_tokens=[int(token[i]) for i in path[1:]], accept_len=len(path) - 1,
                bonus=int(bonus), terminal_rank=int(pr["rank"][path[-1]]))


def verify_step(batch, policy, with_attention=True):
    out = []
    for b in range(len(batch["node_off"]) - 1):
        stats, sc = quantify(batch, policy, b)
        pr = stratify_prune(batch, policy, b, sc)
        res = dict(stats=stats, scores=sc, pruned=pr)
        if with_attention:
            res["attn_out"], res["attn_lse"] = verify_attention(batch, b, pr)
        res["accept"] = accept_path(batch, b, pr)
        out.append(res)
    return out
