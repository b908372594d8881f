"""GPU parity of the exported code paths beyond the five workloads: compacted row layout, head-major KV
cache, the Philox stream by value and the `uniforms` override, the cold paths of the Top-K (heavy ties,
-inf logits, vocabularies that are no multiple of the 16-byte vector), K = 1 and 16, a GQA group of 16,
duplicate sibling tokens, a path longer than the output slots, logits written by the kernel right ahead of
the call.  Every case goes through the C ABI and is compared with the CPU oracle element by element."""
import numpy as np
import pytest
import torch

from oracle import philox as ophilox
from oracle import step as ostep
from paper_2505_13254_b200 import binding as hb
from paper_2505_13254_b200 import step as gstep
from paper_2505_13254_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu

C2S = synth.CONFIGS["c2_8b"].scaled(kv_len=(333, 333))
C3S = synth.CONFIGS["c3_70b"].scaled(kv_len=(200, 200))
C4S = synth.CONFIGS["c4_ragged"].scaled(batch=5, kv_len=(1, 400))


@pytest.fixture(scope="module")
def ctx():
    c = hb.Context(0, 256 << 20)
    yield c
    c.close()


def check_all(st, batch, res, policy, attention=True, compact=False):
    torch.cuda.synchronize()
    pu.check_quant(st.quant, batch, res, policy["top_k"])
    pu.check_pruned(st.pruned, res)
    if attention:
        pu.check_attention(st.attn_out, st.attn_lse, batch, res, compact=compact)
    pu.check_accept(st.accept, res)


# ---- (i) compacted rows: q, k_tree, v_tree, out and the target logits indexed by kept node -----------------

@pytest.mark.parametrize("cfg,base,seed", [(C2S, "c2_8b", 1100), (C3S, "c3_70b", 1200), (C4S, "c4_ragged", 1300),
                                           (C4S.scaled(accept="mixed3", batch=6), "c4_ragged", 1400)])
def test_compact_row_layout(ctx, cfg, base, seed):
    policy = pu.policy_for(cfg, base)
    batch, res = pu.oracle_case(cfg, policy, seed)
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy)
    st.quantify(db)
    st.prune(db)
    keep = torch.cat([torch.from_numpy(batch["node_off"][b] + r["pruned"]["keep_idx"]) for b, r in enumerate(res)]).cuda()
    q, kt, vt, tgt = (t.index_select(0, keep).contiguous() for t in (db.q, db.k_tree, db.v_tree, db.target))
    out, lse = torch.zeros_like(q), torch.zeros(q.shape[0], q.shape[1], dtype=torch.float32, device=q.device)
    hb.hs_tree_verify_attention(ctx, st.pruned, q, kt, vt, db.k_cache, db.v_cache, db.kv_off, batch=db.tree.batch,
                                max_nodes=db.max_nodes, max_kv_len=db.max_kv_len, layout=hb.HS_ROWS_COMPACT,
                                out=out, lse_out=lse)
    hb.hs_accept_path(ctx, db.tree, st.pruned, tgt, db.draft if db.any_sampling else None, db.mode, db.temperature,
                      target_layout=hb.HS_ROWS_COMPACT, seed=db.seed, offset=db.offset, out=st.accept)
    st.attn_out, st.attn_lse = out, lse
    check_all(st, batch, res, policy, compact=True)
    assert hb.hs_device_error(ctx) == 0


# ---- (ii) head-major KV cache: [hkv][tokens][128] memory behind the same [tokens, hkv, 128] view -------------

@pytest.mark.parametrize("cfg,base,seed", [(C2S, "c2_8b", 1500), (C4S, "c4_ragged", 1600)])
def test_head_major_kv_cache(ctx, cfg, base, seed):
    policy = pu.policy_for(cfg, base)
    batch, res = pu.oracle_case(cfg, policy, seed)
    db = gstep.upload(batch)
    db.k_cache = db.k_cache.permute(1, 0, 2).contiguous().permute(1, 0, 2)
    db.v_cache = db.v_cache.permute(1, 0, 2).contiguous().permute(1, 0, 2)
    assert db.k_cache.stride(1) > db.k_cache.stride(0)
    st = gstep.VerifyStep(ctx, db, policy).run(db)
    check_all(st, batch, res, policy)
    assert hb.hs_device_error(ctx) == 0


# ---- (iii) the Philox stream by value, offsets, and the uniforms override ----------------------------------

def test_philox_words_match_the_oracle_stream(ctx):
    rng = np.random.default_rng(5)
    n = 400
    b = rng.integers(0, 4096, n).astype(np.int32)
    node = rng.integers(0, 128, n).astype(np.int32)
    sid = rng.integers(0, 2, n).astype(np.int32)
    dev = lambda a: torch.from_numpy(a).cuda()
    for seed, offset in ((0, 0), (0x1234567, 0), (0x9E3779B97F4A7C15, 77), (0xDEADBEEF00000001, (3 << 32) + 5),
                         ((1 << 64) - 1, (1 << 63) - 1)):
        got = hb.hs_philox_uniforms(ctx, seed, offset, dev(b), dev(node), dev(sid)).cpu().numpy()
        want = np.array([ophilox.uniform(seed, offset, int(b[i]), int(node[i]), int(sid[i])) for i in range(n)])
        assert np.array_equal(got.astype(np.float64), want), (hex(seed), offset)
    with pytest.raises(hb.HsError):
        hb.hs_philox_uniforms(ctx, 1, 1 << 63, dev(b), dev(node), dev(sid))


@pytest.mark.parametrize("cfg,base,seed", [(C3S, "c3_70b", 1700), (C4S.scaled(accept="mixed3", batch=6), "c4_ragged", 1800)])
def test_philox_offset_and_uniforms_override(ctx, cfg, base, seed):
    policy = pu.policy_for(cfg, base)
    offset = (5 << 32) + 12345

    def with_offset(batch):
        batch["philox_offset"] = offset
        batch["philox_seed"] |= 1 << 63                   # a seed whose high word matters

    batch, res = pu.oracle_case(cfg, policy, seed, attention="none", mutate=with_offset)
    db = gstep.upload(batch)
    assert db.offset == offset
    st = gstep.VerifyStep(ctx, db, policy).run(db)
    check_all(st, batch, res, policy, attention=False)
    first = [t.clone() for t in (st.accept.accept_len, st.accept.path_nodes, st.accept.path_tokens, st.accept.bonus_token)]
    # the same values handed over as an array give the same walk
    n = db.tree.n_nodes_total
    u = np.zeros(n + cfg.batch, dtype=np.float32)
    for b in range(cfg.batch):
        lo, hi = batch["node_off"][b], batch["node_off"][b + 1]
        for i in range(hi - lo):
            u[lo + i] = ophilox.uniform(batch["philox_seed"], offset, b, i, 0)
        u[n + b] = ophilox.uniform(batch["philox_seed"], offset, b, 0, 1)
    hb.hs_accept_path(ctx, db.tree, st.pruned, db.target, db.draft, db.mode, db.temperature,
                      target_layout=hb.HS_ROWS_ORIGINAL, seed=999, offset=1, uniforms=torch.from_numpy(u).cuda(),
                      out=st.accept)
    torch.cuda.synchronize()
    pu.check_accept(st.accept, res)
    again = (st.accept.accept_len, st.accept.path_nodes, st.accept.path_tokens, st.accept.bonus_token)
    assert all(torch.equal(a, b) for a, b in zip(first, again))


# ---- (iv) cold paths of the vocabulary pass ----------------------------------------------------------------

def hand_batch(draft, parent, token, dtype):
    """A one-sequence batch around hand-made draft rows (float32 values; bf16 rows are rounded first)."""
    draft = np.asarray(draft, dtype=np.float32)
    cfg = synth.CONFIGS["c2_8b"].scaled(vocab=draft.shape[1], logits_dtype=dtype, n_nodes=(len(parent),) * 2)
    stored = synth.f32_to_bf16_bits(draft) if dtype == "bf16" else draft
    n = len(parent)
    return dict(cfg=cfg, node_off=np.array([0, n], dtype=np.int32), kv_off=np.array([0, 0], dtype=np.int32),
                parent=np.asarray(parent, dtype=np.int32), token=np.asarray(token, dtype=np.int32), draft=stored,
                target=stored, mode=np.zeros(1, dtype=np.int32), temperature=np.zeros(1, dtype=np.float32),
                philox_seed=1, philox_offset=0)


def quantify_against_oracle(ctx, batch, policy, padded_stride=None):
    db = gstep.upload(batch)
    if padded_stride:                                          # rows padded to the stride the entry point asks for
        wide = torch.full((db.draft.shape[0], padded_stride), 7.0, dtype=db.draft.dtype, device=db.draft.device)
        wide[:, : db.draft.shape[1]] = db.draft
        db.draft = wide[:, : db.draft.shape[1]]
        assert db.draft.stride(0) == padded_stride
    q = hb.hs_entropy_quantify(ctx, db.tree, db.draft, policy)
    torch.cuda.synchronize()
    stats, sc = ostep.quantify(batch, policy, 0)
    pu.check_quant(q, batch, [dict(stats=stats, scores=sc)], policy["top_k"])
    return q


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_topk_with_heavy_ties_and_minus_infinity(ctx, dtype):
    rng = np.random.default_rng(3)
    V = 128256 if dtype == "bf16" else 50000
    rows = rng.standard_normal((7, V)).astype(np.float32)
    rows[0, :] = 1.25                                          # constant row: every logit ties
    rows[1, :] = -3.0
    rows[1, rng.choice(V, 900, replace=False)] = 2.5           # 900 equal maxima
    rows[2, rng.choice(V, V // 2, replace=False)] = -np.inf    # half of the vocabulary masked out
    rows[3, :] = -np.inf
    rows[3, [5, 77, V - 1]] = [0.5, 0.5, -1.0]                 # fewer finite logits than K
    rows[4, 16384 * 3: 16384 * 3 + 600] = 9.0                  # the ties sit in one chunk of the row
    rows[5, ::2] = 0.0                                         # ties across every chunk
    parent = [-1, 0, 0, 1, 1, 2, 5]
    token = [0, 3, 4, 10, 11, int(np.nonzero(np.isfinite(rows[2]))[0][0]), 13]     # (tokens with finite draft logits)
    batch = hand_batch(rows, parent, token, dtype)
    policy = pu.policy_for(batch["cfg"], "c2_8b")
    q = quantify_against_oracle(ctx, batch, policy)
    assert q.topk_idx[0].tolist() == list(range(policy["top_k"]))      # ties: lowest token ids first
    assert abs(float(q.h_full[0]) - np.log(V)) < 1e-3 and abs(float(q.i_topk[0]) - np.log(policy["top_k"])) < 1e-5


@pytest.mark.parametrize("dtype,vocab,stride", [("bf16", 32003, 32008), ("f32", 32003, 32004), ("bf16", 1001, 1008),
                                                ("f32", 7, 8), ("bf16", 16390, 16392)])
def test_vocabulary_not_a_multiple_of_the_vector(ctx, dtype, vocab, stride):
    rng = np.random.default_rng(vocab)
    rows = (rng.standard_normal((6, vocab)) * 2).astype(np.float32)
    rows[2, vocab - 1] = 30.0                                  # the maximum is the very last token
    parent = [-1, 0, 0, 1, 2, 2]
    token = [0, 1, vocab - 1, 2, vocab - 1, 0]
    batch = hand_batch(rows, parent, token, dtype)
    policy = dict(pu.policy_for(batch["cfg"], "c2_8b"), top_k=min(10, vocab))
    quantify_against_oracle(ctx, batch, policy, padded_stride=stride)


# ---- (v) other K, a GQA group of 16, duplicate sibling tokens, short path output -----------------------------

@pytest.mark.parametrize("top_k", [1, 2, 16])
def test_other_top_k(ctx, top_k):
    policy = dict(pu.policy_for(C2S, "c2_8b"), top_k=top_k)
    if top_k == 16:
        policy["thresholds"] = list(np.linspace(6.0, 20.0, 7))
    batch, res = pu.oracle_case(C2S, policy, 1900 + top_k, attention="none")
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy).run(db)
    check_all(st, batch, res, policy, attention=False)


@pytest.mark.parametrize("hq,hkv", [(32, 2), (16, 1), (48, 8)])
def test_gqa_group_sizes(ctx, hq, hkv):
    cfg = C2S.scaled(hq=hq, hkv=hkv, kv_len=(130, 130))
    policy = pu.policy_for(cfg, "c2_8b")
    batch, res = pu.oracle_case(cfg, policy, 2000 + hq)
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy).run(db)
    check_all(st, batch, res, policy)
    assert hb.hs_device_error(ctx) == 0


def duplicate_sibling_tokens(batch):
    """The second child of every node that has two or more takes the token of the first."""
    for b in range(len(batch["node_off"]) - 1):
        lo, hi = batch["node_off"][b], batch["node_off"][b + 1]
        par = batch["parent"][lo:hi]
        for p in range(hi - lo):
            kids = np.nonzero(par == p)[0]
            if len(kids) >= 2:
                batch["token"][lo + kids[1]] = batch["token"][lo + kids[0]]


@pytest.mark.parametrize("accept", ["greedy", "rejection", "deterministic"])
@pytest.mark.parametrize("seed", [2100, 2101, 2102])
def test_duplicate_sibling_tokens(ctx, accept, seed):
    cfg = C3S.scaled(accept=accept, temperature=1.0 if accept != "greedy" else 0.0)
    policy = pu.policy_for(cfg, "c3_70b")
    batch, res = pu.oracle_case(cfg, policy, seed, attention="none", mutate=duplicate_sibling_tokens)
    lo, hi = batch["node_off"][0], batch["node_off"][1]
    kids0 = np.nonzero(batch["parent"][lo:hi] == 0)[0]
    assert batch["token"][lo + kids0[0]] == batch["token"][lo + kids0[1]]
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy).run(db)
    check_all(st, batch, res, policy, attention=False)


def test_path_longer_than_the_output_slots(ctx):
    cfg = C4S.scaled(accept="mixed3", batch=6)
    policy = pu.policy_for(cfg, "c4_ragged")
    batch, res = pu.oracle_case(cfg, policy, 2200, attention="none")
    assert max(r["accept"]["accept_len"] for r in res) >= 3
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy, path_cap=2).run(db)
    torch.cuda.synchronize()
    for b, r in enumerate(res):
        acc = r["accept"]
        assert int(st.accept.accept_len[b]) == acc["accept_len"] and int(st.accept.bonus_token[b]) == acc["bonus"]
        assert [x for x in st.accept.path_nodes[b].tolist() if x >= 0] == acc["path_nodes"][:2]
        assert [x for x in st.accept.path_tokens[b].tolist() if x >= 0] == acc["path_tokens"][:2]


def test_more_than_64_kept_nodes(ctx):
    """A policy that keeps the whole 96-node tree: the tree keys fill two key tiles of the attention."""
    cfg = synth.CONFIGS["c5_long"].scaled(batch=2, kv_len=(700, 777))
    policy = dict(pu.policy_for(cfg, "c5_long"), n_default=128, d_base=12, alpha=6)
    batch, res = pu.oracle_case(cfg, policy, 2250)
    assert all(len(r["pruned"]["keep_idx"]) == 96 for r in res)
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy).run(db)
    check_all(st, batch, res, policy)
    assert hb.hs_device_error(ctx) == 0


# ---- logits written by the kernel directly ahead of the call (no early read of caller inputs by default) ------

def test_logits_written_by_the_preceding_kernel(ctx):
    policy = pu.policy_for(C2S, "c2_8b")
    batch, res = pu.oracle_case(C2S, policy, 2300, attention="none")
    db = gstep.upload(batch)
    good = db.draft.clone()
    junk = torch.randn(good.shape, device=good.device).to(good.dtype)
    st = gstep.VerifyStep(ctx, db, policy)
    for _ in range(20):
        db.draft.copy_(junk)
        torch.add(good, 0, out=db.draft)                       # an elementwise kernel writes the rows ...
        st.quantify(db)                                        # ... and the pass follows it in the stream
        st.prune(db)
        torch.cuda.synchronize()
        pu.check_quant(st.quant, batch, res, policy["top_k"])
        pu.check_pruned(st.pruned, res)


def test_prefetch_flags_give_the_same_results(ctx):
    policy = pu.policy_for(C2S, "c2_8b")
    batch, res = pu.oracle_case(C2S, policy, 2400)
    db = gstep.upload(batch)
    try:
        hb.hs_set_prefetch(ctx, hb.HS_PREFETCH_LOGITS | hb.HS_PREFETCH_KV)
        st = gstep.VerifyStep(ctx, db, policy).run(db)
        check_all(st, batch, res, policy)
    finally:
        hb.hs_set_prefetch(ctx, 0)
    with pytest.raises(hb.HsError):
        hb.hs_set_prefetch(ctx, 64)


# ---- (viii) every entropy bin ----------------------------------------------------------------------------------

def test_every_bin_occurs_and_matches(ctx):
    cfg = C2S.scaled(kv_len=(64, 64))
    pol = pu.policy_for(cfg, "c2_8b")
    bins = set()
    for seed in range(3000, 3060):
        batch, res = pu.oracle_case(cfg, pol, seed * 50, attention="none")
        db = gstep.upload(batch)
        st = gstep.VerifyStep(ctx, db, pol).run(db)
        check_all(st, batch, res, pol, attention=False)
        bins.add(res[0]["pruned"]["bin"])
        if len(bins) == 8:
            break
    assert bins == set(range(8))


# ---- the fused call (entropy pass, then tree scores + pruning in one kernel) against the two separate calls -------

@pytest.mark.parametrize("batch,seed,nodes", [(1, 2600, (3, 60)), (7, 2601, (3, 60)), (40, 2602, (3, 60)),
                                              (150, 2603, (3, 60)), (3000, 2604, (2, 6))])
def test_fused_quantify_prune_equals_the_two_calls(ctx, batch, seed, nodes):
    """The CTAs of the fused kernel hand their kept counts to one another (the offsets of the compacted arrays).
    With 3000 sequences there are more CTAs than the device holds at once: a CTA only waits for lower-numbered
    ones, which were started before it.  Twice in a row: the hand-over flags have put themselves back."""
    cfg = synth.CONFIGS["c4_ragged"].scaled(batch=batch, vocab=4096 if batch < 1000 else 512, n_nodes=nodes)
    policy = pu.policy_for(cfg, "c4_ragged")
    batch_np = synth.make_batch(cfg, seed, with_attention=False)
    db = gstep.upload(batch_np)
    two = gstep.VerifyStep(ctx, db, policy)
    two.quantify(db)
    two.prune(db)
    one = gstep.VerifyStep(ctx, db, policy)
    for rep in range(2):
        for t in (one.pruned.keep_idx, one.pruned.keep_off, one.pruned.n_keep, one.quant.phi):
            t.fill_(-7)
        one.quantify_prune(db)
        torch.cuda.synchronize()
        for name in ("row_max", "row_lse", "h_full", "i_topk", "topk_idx", "logc", "score", "phi", "depth", "pstar_node",
                     "phi_star", "status"):
            assert torch.equal(getattr(one.quant, name), getattr(two.quant, name)), name
        total = int(two.pruned.keep_off[-1])
        assert torch.equal(one.pruned.keep_off, two.pruned.keep_off) and torch.equal(one.pruned.n_keep, two.pruned.n_keep)
        for name in ("keep_idx", "new_parent", "new_depth", "keep_rank", "anc_mask"):
            assert torch.equal(getattr(one.pruned, name)[:total], getattr(two.pruned, name)[:total]), name
        for name in ("bin", "d_prime", "n_prime", "status"):
            assert torch.equal(getattr(one.pruned, name), getattr(two.pruned, name)), name
    assert hb.hs_device_error(ctx) == 0
