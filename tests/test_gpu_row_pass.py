"""hs_accept_path reads the vocabulary rows with one of two kernels (hs_set_row_pass): small CTAs that own one
32 KiB chunk of a row, or one persistent CTA per SM that streams its share of all rows.  The default picks by the
size of the launch, so the small parity cases never reach the streaming kernel by themselves: here every
acceptance case runs with each kernel forced and is compared with the CPU oracle (bit-exact paths, bonus tokens
and ranks), including ragged vocabularies, fp32 logits, empty and malformed sequences, compacted target rows."""
import numpy as np
import pytest
import torch

from paper_2505_13254_b200 import binding as hb
from paper_2505_13254_b200 import step as gstep
from paper_2505_13254_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu

VARIANTS = {"chunk": hb.HS_ROW_PASS_CHUNK, "stream": hb.HS_ROW_PASS_STREAM}


@pytest.fixture(scope="module", params=sorted(VARIANTS))
def ctx(request):
    c = hb.Context(0, 256 << 20)
    hb.hs_set_row_pass(c, VARIANTS[request.param])
    yield c
    c.close()


CASES = {
    "c1_f32_greedy": (synth.CONFIGS["c1_tiny"], "c1_tiny"),
    "c2_bf16_greedy": (synth.CONFIGS["c2_8b"], "c2_8b"),
    "c3_rejection": (synth.CONFIGS["c3_70b"], "c3_70b"),
    "c3_deterministic": (synth.CONFIGS["c3_70b"].scaled(accept="deterministic"), "c3_70b"),
    "c4_mixed": (synth.CONFIGS["c4_ragged"].scaled(batch=7), "c4_ragged"),
    "c4_mixed3": (synth.CONFIGS["c4_ragged"].scaled(batch=9, accept="mixed3"), "c4_ragged"),
    "c5_rejection_T07": (synth.CONFIGS["c5_long"].scaled(batch=3), "c5_long"),
    "c4_f32_mixed3": (synth.CONFIGS["c4_ragged"].scaled(batch=5, accept="mixed3", logits_dtype="f32", vocab=50000), "c4_ragged"),
}


def run_accept(ctx, db, policy, **kw):
    st = gstep.VerifyStep(ctx, db, policy, **kw)
    st.quantify(db)
    st.prune(db)
    st.accept_path(db)
    torch.cuda.synchronize()
    return st


@pytest.mark.parametrize("name", sorted(CASES))
@pytest.mark.parametrize("seed", [3100, 3200])
def test_acceptance_matches_the_oracle(ctx, name, seed):
    cfg, base = CASES[name]
    policy = pu.policy_for(cfg, base)
    batch, res = pu.oracle_case(cfg, policy, seed, attention="none")
    db = gstep.upload(batch)
    st = run_accept(ctx, db, policy)
    pu.check_pruned(st.pruned, res)
    pu.check_accept(st.accept, res)
    first = [t.clone() for t in (st.accept.path_nodes, st.accept.path_tokens, st.accept.bonus_token, st.accept.accept_len)]
    st.accept_path(db)                          # the arrival counters have reset themselves
    torch.cuda.synchronize()
    pu.check_accept(st.accept, res)
    assert all(torch.equal(a, b) for a, b in zip(first, (st.accept.path_nodes, st.accept.path_tokens,
                                                         st.accept.bonus_token, st.accept.accept_len)))
    assert hb.hs_device_error(ctx) == 0


def padded(t, stride, fill):
    """The same rows behind a wider row stride; what lies between the rows is `fill`."""
    wide = torch.full((t.shape[0], stride), fill, dtype=t.dtype, device=t.device)
    wide[:, : t.shape[1]] = t
    return wide[:, : t.shape[1]]


@pytest.mark.parametrize("dtype,vocab,stride", [("bf16", 32003, 32008), ("f32", 32003, 32004), ("bf16", 16385, 16392),
                                                ("bf16", 70001, 70016)])
@pytest.mark.parametrize("accept", ["greedy", "mixed3"])
def test_vocabulary_not_a_multiple_of_the_vector(ctx, dtype, vocab, stride, accept):
    cfg = synth.CONFIGS["c4_ragged"].scaled(batch=4, vocab=vocab, logits_dtype=dtype, accept=accept)
    policy = pu.policy_for(cfg, "c4_ragged")
    batch, res = pu.oracle_case(cfg, policy, 3300, attention="none")
    db = gstep.upload(batch)
    db.draft = padded(db.draft, stride, 60.0)   # larger than every logit: a read past the vocabulary would win
    db.target = padded(db.target, stride, 60.0)
    st = run_accept(ctx, db, policy)
    pu.check_pruned(st.pruned, res)
    pu.check_accept(st.accept, res)


def test_compacted_target_rows(ctx):
    cfg = synth.CONFIGS["c4_ragged"].scaled(batch=6, accept="mixed3")
    policy = pu.policy_for(cfg, "c4_ragged")
    batch, res = pu.oracle_case(cfg, policy, 3400, attention="none")
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy)
    st.quantify(db)
    st.prune(db)
    keep = torch.cat([torch.from_numpy(batch["node_off"][b] + r["pruned"]["keep_idx"]) for b, r in enumerate(res)]).cuda()
    tgt = db.target.index_select(0, keep).contiguous()
    hb.hs_accept_path(ctx, db.tree, st.pruned, tgt, db.draft, db.mode, db.temperature, target_layout=hb.HS_ROWS_COMPACT,
                      seed=db.seed, offset=db.offset, out=st.accept)
    torch.cuda.synchronize()
    pu.check_accept(st.accept, res)


@pytest.mark.parametrize("bad", [0, 2, 4])
def test_flagged_and_empty_sequences(ctx, bad):
    cfg = synth.CONFIGS["c4_ragged"].scaled(batch=5, n_nodes=(20, 60), accept="mixed3")
    policy = pu.policy_for(cfg, "c4_ragged")
    batch, res = pu.oracle_case(cfg, policy, 3500, attention="none")
    db = gstep.upload(batch)
    lo = int(batch["node_off"][bad])
    db.tree.parent[lo + 3] = 7                  # a parent that comes after its child: the sequence is flagged upstream
    st = run_accept(ctx, db, policy)
    assert int(st.accept.status[bad]) == hb.HS_ERR_BAD_TREE and int(st.accept.accept_len[bad]) == 0
    assert int(st.accept.bonus_token[bad]) == -1 and (st.accept.path_nodes[bad] == -1).all()
    healthy = [r if b != bad else None for b, r in enumerate(res)]
    pu.check_pruned(st.pruned, healthy)
    pu.check_accept(st.accept, healthy)
    # rejection mode without draft logits: an error of that sequence alone
    acc = hb.hs_accept_path(ctx, db.tree, st.pruned, db.target, None, db.mode, db.temperature,
                            target_layout=hb.HS_ROWS_ORIGINAL, seed=db.seed, offset=db.offset)
    torch.cuda.synchronize()
    for b in range(cfg.batch):
        if b == bad:
            assert int(acc.status[b]) == hb.HS_ERR_BAD_TREE
        elif batch["mode"][b] == hb.HS_ACCEPT_REJECTION:
            assert int(acc.status[b]) == hb.HS_ERR_INVALID_ARG and int(acc.accept_len[b]) == 0
        else:
            assert int(acc.status[b]) == 0 and int(acc.accept_len[b]) == res[b]["accept"]["accept_len"]
    assert hb.hs_device_error(ctx) == 0


def test_the_knob_refuses_unknown_variants(ctx):
    with pytest.raises(hb.HsError):
        hb.hs_set_row_pass(ctx, 3)
    with pytest.raises(hb.HsError):
        hb.hs_set_row_pass(ctx, -1)
