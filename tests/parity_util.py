"""Shared helpers of the GPU parity tests: guard-banded cases and element-wise comparisons."""
import json
import os

import numpy as np

from oracle import step as ostep
from oracle import tree as otree
from paper_2505_13254_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
THRESHOLDS = json.load(open(os.path.join(GOLD, "thresholds.json")))

# guard bands of the float -> integer decisions (the GPU decides in fp32, the oracle in fp64)
BAND_BIN, BAND_RANK, BAND_PSTAR, BAND_ACCEPT, BAND_CDF = 1e-3, 1e-4, 1e-4, 1e-4, 5e-7


def policy_for(cfg, base=None):
    name = base or cfg.name
    return synth.default_policy(cfg, THRESHOLDS[name]["thresholds"])


def _sequence_ok(batch, policy, b):
    """Oracle results of sequence b, or None if one of its float decisions is inside a guard band."""
    stats, sc = ostep.quantify(batch, policy, b)
    m = otree.margins(sc, policy)
    if m["bin"] <= BAND_BIN or m["rank"] <= BAND_RANK or m["pstar"] <= BAND_PSTAR:
        return None
    pr = ostep.stratify_prune(batch, policy, b, sc)
    trace = []
    acc = ostep.accept_path(batch, b, pr, trace=trace)
    for t in trace:
        if t[0] == "accept" and abs(t[2] - t[3]) <= BAND_ACCEPT:
            return None
        if t[0] == "final" and (t[1] - t[2] <= BAND_CDF or t[3] - t[1] <= BAND_CDF):
            return None
    return dict(stats=stats, scores=sc, pruned=pr, accept=acc)


def systematic_pairs(nk, hq, hkv, block=128, tile=64):
    """(node, query head) pairs that cover the attention kernel's structure: with query rows numbered
    node * G + g (G = hq / hkv), the first and the last row of every block of `block` rows under every
    key/value head, plus the kept nodes on both sides of every `tile`-key boundary of the tree keys and the
    last node (their tree columns straddle a key tile)."""
    g_sz = hq // hkv
    rows = nk * g_sz
    pairs = set()
    for r0 in range(0, rows, block):
        for r in (r0, min(r0 + block, rows) - 1):
            node, g = divmod(r, g_sz)
            for h in range(hkv):
                pairs.add((node, h * g_sz + g))
    for node in {nk - 1, 0} | {j for t in range(tile, nk, tile) for j in (t - 1, t)}:
        for h in range(hkv):
            pairs.add((node, h * g_sz + (node % g_sz)))
    return sorted(pairs)


def oracle_case(cfg, policy, seed, attention="full", attn_pairs=64, max_tries=20, mutate=None):
    """Generates a batch whose every float decision keeps its guard band (a sequence that does
    not is re-drawn alone with the next salt) and runs the oracle on it.
    attention: "full" | "sampled" (random pairs) | "systematic" (systematic_pairs + random pairs) | "none".
    mutate(batch): optional in-place edit of the generated batch (before the oracle sees it)."""
    salts = [0] * cfg.batch
    res = [None] * cfg.batch
    for _ in range(max_tries):
        probe = synth.make_batch(cfg, seed, with_attention=False, salts=salts)
        if mutate:
            mutate(probe)
        for b in range(cfg.batch):
            if res[b] is None:
                res[b] = _sequence_ok(probe, policy, b)
                if res[b] is None:
                    salts[b] += 1
        if all(r is not None for r in res):
            break
    else:
        raise RuntimeError("no guard-banded draw found")
    batch = synth.make_batch(cfg, seed, with_attention=attention != "none", salts=salts)
    if mutate:
        mutate(batch)
    if attention != "none":
        rng = np.random.default_rng(seed)
        for b, r in enumerate(res):
            nk = len(r["pruned"]["keep_idx"])
            pairs = None
            if attention in ("sampled", "systematic"):
                pairs = [(int(rng.integers(nk)), int(rng.integers(cfg.hq))) for _ in range(attn_pairs)]
                pairs += [(nk - 1, h) for h in range(0, cfg.hq, max(1, cfg.hq // 8))]
                if attention == "systematic":
                    pairs = sorted(set(pairs) | set(systematic_pairs(nk, cfg.hq, cfg.hkv)))
            r["attn_out"], r["attn_lse"] = ostep.verify_attention(batch, b, r["pruned"], rows=pairs)
    return batch, res


def rel_close(got, want, rel=1e-4, abs_=1e-6):
    """|got - want| <= rel * |want| + abs_.  The absolute term covers values that are exactly or nearly 0
    (the entropy of a one-hot row, ln c of a token with probability 1), where a relative bound is void."""
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    return np.all(np.abs(got - want) <= rel * np.abs(want) + abs_), float(np.max(np.abs(got - want) / (np.abs(want) + abs_ / rel)))


def check_quant(q, batch, res, K):
    """Entropies within 1e-4 relative; maxima, Top-K ids and values, depths and P* exact."""
    node_off = batch["node_off"]
    for b, r in enumerate(res):
        if r is None:                                # a sequence the test made invalid: checked by its status
            continue
        lo, hi = node_off[b], node_off[b + 1]
        st = r["stats"]
        assert np.array_equal(q.row_max[lo:hi].cpu().numpy().astype(np.float64), [s["max"] for s in st])
        for name, key in (("row_lse", "lse"), ("h_full", "H"), ("i_topk", "I_topk"), ("i_trunc", "I_trunc")):
            ok, err = rel_close(getattr(q, name)[lo:hi].cpu().numpy(), [s[key] for s in st])
            assert ok, (name, b, err)
        want_val, want_idx = np.stack([s["topk_val"] for s in st]), np.stack([s["topk_idx"] for s in st])
        got_idx = q.topk_idx[lo:hi].cpu().numpy()
        assert np.array_equal(q.topk_val[lo:hi].cpu().numpy().astype(np.float64), want_val)
        # a row with fewer than K finite logits: the slots past them hold -inf and token id -1
        fin = np.isfinite(want_val)
        assert np.array_equal(got_idx[fin], want_idx[fin]) and (got_idx[~fin] == -1).all()
        sc = r["scores"]
        for name, key in (("logc", "logc"), ("score", "S"), ("phi", "Phi")):
            ok, err = rel_close(getattr(q, name)[lo:hi].cpu().numpy(), sc[key], abs_=1e-5)
            assert ok, (name, b, err)
        assert np.array_equal(q.depth[lo:hi].cpu().numpy(), sc["depth"])
        assert int(q.pstar_node[b]) == sc["pstar_node"]
        ok, err = rel_close(float(q.phi_star[b]), sc["phi_star"], abs_=1e-5)
        assert ok, ("phi_star", b, err)
        assert int(q.status[b]) == 0


def check_pruned(p, res):
    """Bit-exact: bins, d', N', kept node sets, parents, depths, ranks and ancestor masks."""
    off = p.keep_off.cpu().numpy()
    for b, r in enumerate(res):
        if r is None:
            continue
        pr = r["pruned"]
        nk = len(pr["keep_idx"])
        assert (int(p.bin[b]), int(p.d_prime[b]), int(p.n_prime[b]), int(p.n_keep[b])) == \
            (pr["bin"], pr["d_prime"], pr["n_prime"], nk)
        assert off[b + 1] - off[b] == nk
        sl = slice(off[b], off[b + 1])
        assert np.array_equal(p.keep_idx[sl].cpu().numpy(), pr["keep_idx"])
        assert np.array_equal(p.new_parent[sl].cpu().numpy(), pr["new_parent"])
        assert np.array_equal(p.new_depth[sl].cpu().numpy(), pr["new_depth"])
        assert np.array_equal(p.keep_rank[sl].cpu().numpy(), pr["rank"])
        words = p.anc_mask[sl].cpu().numpy().view(np.uint64)
        want = np.zeros((nk, 2), dtype=np.uint64)
        for i in range(nk):
            for j in np.nonzero(pr["mask"][i])[0]:
                want[i, j // 64] |= np.uint64(1) << np.uint64(j % 64)
        assert np.array_equal(words, want)


def check_accept(a, res):
    """Bit-exact: accepted length, path (original and compact ids), tokens, bonus token, rank.  A path
    longer than the output's path_cap is compared on the slots that exist."""
    cap = a.path_cap
    for b, r in enumerate(res):
        if r is None:
            continue
        acc = r["accept"]
        n = acc["accept_len"]
        assert int(a.status[b]) == 0
        assert int(a.accept_len[b]) == n, (b, int(a.accept_len[b]), n)
        assert a.path_nodes[b, : n + 1].tolist() == acc["path_nodes"][:cap]
        assert a.path_compact[b, : n + 1].tolist() == acc["path_compact"][:cap]
        assert a.path_tokens[b, :n].tolist() == acc["path_tokens"][:cap]
        assert (a.path_nodes[b, n + 1:] == -1).all() and (a.path_tokens[b, n:] == -1).all()
        assert int(a.bonus_token[b]) == acc["bonus"], (b, int(a.bonus_token[b]), acc["bonus"])
        assert int(a.terminal_rank[b]) == acc["terminal_rank"]


def check_attention(out, lse, batch, res, tol=1e-2, compact=False):
    """bf16 output of the kernels against the fp64 oracle: max absolute error <= tol on every
    (node, head) the oracle evaluated; rows are laid out by drafted node id, or compacted
    (kept node i of sequence b in row keep_off[b] + i) with compact=True."""
    node_off = batch["node_off"]
    worst = 0.0
    o = out.float().cpu().numpy().astype(np.float64)
    l = lse.cpu().numpy().astype(np.float64)
    koff = 0
    for b, r in enumerate(res):
        if r is None:
            continue
        nk = len(r["pruned"]["keep_idx"])
        rows = (koff + np.arange(nk)) if compact else node_off[b] + r["pruned"]["keep_idx"]
        koff += nk
        want, want_lse = r["attn_out"], r["attn_lse"]
        got, got_lse = o[rows], l[rows]
        done = ~np.isnan(want[..., 0])
        assert done.any()
        err = np.abs(got[done] - want[done]).max()
        worst = max(worst, err)
        assert err <= tol, (b, err)
        assert np.abs(got_lse[done] - want_lse[done]).max() <= 1e-3 * max(1.0, np.abs(want_lse[done]).max())
    return worst
