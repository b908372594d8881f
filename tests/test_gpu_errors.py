"""Failure handling, injected on the host: malformed trees and out-of-range tokens must end as a per-sequence
status (never a trap) while the healthy sequences of the same batch still match the oracle; bad arguments must
be refused synchronously; a bounded device-side wait that runs out must surface as HS_ERR_TIMEOUT through
hs_device_error and leave the context usable."""
import numpy as np
import pytest
import torch

from paper_2505_13254_b200 import binding as hb
from paper_2505_13254_b200 import step as gstep
from paper_2505_13254_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu

CFG = synth.CONFIGS["c4_ragged"].scaled(batch=5, n_nodes=(20, 60), kv_len=(1, 300), accept="mixed3")


@pytest.fixture(scope="module")
def ctx():
    c = hb.Context(0, 256 << 20)
    yield c
    c.close()


@pytest.fixture(scope="module")
def case():
    policy = pu.policy_for(CFG, "c4_ragged")
    batch, res = pu.oracle_case(CFG, policy, 4100)
    return policy, batch, res


def corrupt(name):
    def forward_parent(db, lo, hi):
        db.tree.parent[lo + 3] = 7                       # points at a later node
    def self_parent(db, lo, hi):
        db.tree.parent[lo + 5] = 5
    def two_roots(db, lo, hi):
        db.tree.parent[lo + 4] = -1
    def rooted_elsewhere(db, lo, hi):
        db.tree.parent[lo] = 0                           # node 0 must be the root
    def token_too_large(db, lo, hi):
        db.tree.token[lo + 2] = CFG.vocab
    def token_negative(db, lo, hi):
        db.tree.token[lo + 2] = -5
    return locals()[name]


@pytest.mark.parametrize("how", ["forward_parent", "self_parent", "two_roots", "rooted_elsewhere", "token_too_large",
                                 "token_negative"])
@pytest.mark.parametrize("bad", [0, 1, 3])
def test_malformed_sequence_is_flagged_and_the_others_still_match(ctx, case, how, bad):
    policy, batch, res = case
    db = gstep.upload(batch)
    lo, hi = int(batch["node_off"][bad]), int(batch["node_off"][bad + 1])
    corrupt(how)(db, lo, hi)
    st = gstep.VerifyStep(ctx, db, policy)
    st.accept.accept_len.fill_(99)
    st.run(db)
    torch.cuda.synchronize()
    assert int(st.quant.status[bad]) == hb.HS_ERR_BAD_TREE and int(st.pruned.status[bad]) == hb.HS_ERR_BAD_TREE
    assert int(st.pruned.n_keep[bad]) == 0 and int(st.accept.accept_len[bad]) == 0
    assert int(st.accept.status[bad]) == hb.HS_ERR_BAD_TREE and int(st.accept.bonus_token[bad]) == -1
    assert (st.accept.path_nodes[bad] == -1).all() and (st.accept.path_tokens[bad] == -1).all()
    healthy = [r if b != bad else None for b, r in enumerate(res)]
    pu.check_quant(st.quant, batch, healthy, policy["top_k"])
    pu.check_pruned(st.pruned, healthy)
    pu.check_attention(st.attn_out, st.attn_lse, batch, healthy)
    pu.check_accept(st.accept, healthy)
    assert hb.hs_device_error(ctx) == 0                  # nothing waited in vain, nothing trapped


def test_sequence_larger_than_the_node_limit_and_empty_sequence(ctx):
    dev = torch.device("cuda:0")
    i32 = lambda a: torch.tensor(a, dtype=torch.int32, device=dev)
    n_big = hb.HS_MAX_NODES + 1
    # three sequences: a chain of 4, an empty one, a star of 129 nodes
    node_off = [0, 4, 4, 4 + n_big]
    parent = [-1, 0, 1, 2] + [-1] + [0] * (n_big - 1)
    token = [0, 1, 2, 3] + [0] * n_big
    tree = hb.TreeBatch(i32(node_off), i32(parent), i32(token), 3, node_off[-1])
    logits = torch.randn(node_off[-1], 512, device=dev)
    policy = dict(thresholds=list(np.linspace(1, 7, 7)), d_base=4, alpha=2, n_default=20, top_k=4,
                  gamma_pct=[30, 60, 100], phi_mode=0, pstar_mode=0, entropy_mode=0)
    q = hb.hs_entropy_quantify(ctx, tree, logits, policy)
    pr = hb.hs_stratify_prune(ctx, tree, q, policy)
    mode = i32([0, 0, 0])
    acc = hb.hs_accept_path(ctx, tree, pr, logits, None, mode, torch.zeros(3, device=dev),
                            target_layout=hb.HS_ROWS_ORIGINAL)
    torch.cuda.synchronize()
    assert q.status.tolist() == [0, hb.HS_ERR_BAD_TREE, hb.HS_ERR_BAD_TREE]
    assert pr.n_keep.tolist()[1:] == [0, 0] and int(pr.n_keep[0]) == 4
    assert pr.keep_off.tolist() == [0, 4, 4, 4]
    assert acc.accept_len.tolist()[1:] == [0, 0] and acc.status.tolist()[1:] == [hb.HS_ERR_BAD_TREE] * 2
    assert int(acc.status[0]) == 0
    assert hb.hs_device_error(ctx) == 0


def test_bad_arguments_are_refused_before_any_launch(ctx, case):
    policy, batch, res = case
    db = gstep.upload(batch)
    status = lambda fn: pytest.raises(hb.HsError, fn).value.status

    unsorted = dict(policy, thresholds=policy["thresholds"][::-1])
    assert status(lambda: hb.hs_entropy_quantify(ctx, db.tree, db.draft, unsorted)) == hb.HS_ERR_INVALID_ARG
    assert status(lambda: hb.hs_entropy_quantify(ctx, db.tree, db.draft, dict(policy, top_k=17))) == hb.HS_ERR_INVALID_ARG
    assert status(lambda: hb.hs_entropy_quantify(ctx, db.tree, db.draft, dict(policy, top_k=0))) == hb.HS_ERR_INVALID_ARG
    # rows that do not start on a 16-byte boundary, a stride that is no multiple of the vector
    flat = torch.zeros(db.draft.numel() + 64, dtype=db.draft.dtype, device=db.draft.device)
    off1 = flat[1: 1 + db.draft.numel()].view_as(db.draft)
    assert status(lambda: hb.hs_entropy_quantify(ctx, db.tree, off1, policy)) == hb.HS_ERR_INVALID_ARG
    odd = torch.zeros(db.draft.shape[0], db.draft.shape[1] + 3, dtype=db.draft.dtype, device=db.draft.device)
    assert status(lambda: hb.hs_entropy_quantify(ctx, db.tree, odd[:, : db.draft.shape[1]], policy)) == hb.HS_ERR_INVALID_ARG
    # a context whose workspace is too small for the batch
    small = hb.Context(0, (256 << 10) + 4096)
    assert status(lambda: hb.hs_entropy_quantify(small, db.tree, db.draft, policy)) == hb.HS_ERR_WORKSPACE
    small.close()
    with pytest.raises(hb.HsError) as e:
        hb.Context(0, 1024)
    assert e.value.status == hb.HS_ERR_WORKSPACE

    st = gstep.VerifyStep(ctx, db, policy)
    st.quantify(db)
    st.prune(db)
    q17 = torch.zeros(db.q.shape[0], 34, 128, dtype=torch.bfloat16, device=db.q.device)
    k2 = db.k_tree[:, :2].contiguous()
    attn = lambda **kw: hb.hs_tree_verify_attention(ctx, st.pruned, kw.get("q", db.q), kw.get("k", db.k_tree),
                                                    kw.get("k", db.v_tree), db.k_cache, db.v_cache, db.kv_off,
                                                    batch=db.tree.batch, max_nodes=kw.get("max_nodes", db.max_nodes),
                                                    max_kv_len=db.max_kv_len, layout=kw.get("layout", hb.HS_ROWS_ORIGINAL),
                                                    node_off=kw.get("node_off", db.tree.node_off))
    assert status(lambda: attn(q=q17, k=k2)) == hb.HS_ERR_SHAPE                       # 17 query heads per kv head
    assert status(lambda: attn(max_nodes=hb.HS_MAX_NODES + 1)) == hb.HS_ERR_INVALID_ARG
    assert status(lambda: attn(node_off=None)) == hb.HS_ERR_INVALID_ARG              # needed for rows by node id
    assert status(lambda: attn(layout=5)) == hb.HS_ERR_INVALID_ARG
    bad_mode_out = hb.AcceptOut(db.tree.batch, 1, db.q.device)
    assert status(lambda: hb.hs_accept_path(ctx, db.tree, st.pruned, db.target, None, db.mode, db.temperature,
                                            target_layout=hb.HS_ROWS_ORIGINAL, out=bad_mode_out)) == hb.HS_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert hb.hs_device_error(ctx) == 0


def test_rejection_mode_without_draft_logits_is_a_per_sequence_error(ctx, case):
    policy, batch, res = case
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy)
    st.quantify(db)
    st.prune(db)
    acc = hb.hs_accept_path(ctx, db.tree, st.pruned, db.target, None, db.mode, db.temperature,
                            target_layout=hb.HS_ROWS_ORIGINAL, seed=db.seed, offset=db.offset)
    torch.cuda.synchronize()
    for b in range(CFG.batch):
        if batch["mode"][b] == hb.HS_ACCEPT_REJECTION:
            assert int(acc.status[b]) == hb.HS_ERR_INVALID_ARG and int(acc.accept_len[b]) == 0
            assert (acc.path_nodes[b] == -1).all() and (acc.path_tokens[b] == -1).all()
        else:
            assert int(acc.status[b]) == 0 and int(acc.accept_len[b]) == res[b]["accept"]["accept_len"]


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(ctx, case):
    policy, batch, res = case
    assert hb.hs_device_error(ctx) == 0
    hb.hs_selftest_wait_timeout(ctx, 200_000)            # nothing completes that barrier: gives up after 0.2 ms
    assert hb.hs_device_error(ctx) == hb.HS_ERR_TIMEOUT
    assert hb.hs_device_error(ctx) == 0                  # read and cleared
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy).run(db)
    torch.cuda.synchronize()
    pu.check_pruned(st.pruned, res)
    pu.check_accept(st.accept, res)
    assert hb.hs_device_error(ctx) == 0
