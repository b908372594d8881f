"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element, on the
same seeded inputs.  Integer outputs are bit-exact; entropies 1e-4 relative; attention 1e-2 absolute."""
import numpy as np
import pytest
import torch

from paper_2505_13254_b200 import binding as hb
from paper_2505_13254_b200 import step as gstep
from paper_2505_13254_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = hb.Context(0, 768 << 20)
    yield c
    c.close()


def run_and_check(ctx, cfg, policy, seed, attention="full", **kw):
    batch, res = pu.oracle_case(cfg, policy, seed, attention=attention, **kw)
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy)
    for rep in range(2):                       # twice: outputs must be bit-identical run to run
        st.run(db)
        torch.cuda.synchronize()
        pu.check_quant(st.quant, batch, res, policy["top_k"])
        pu.check_pruned(st.pruned, res)
        if attention != "none":
            pu.check_attention(st.attn_out, st.attn_lse, batch, res)
        pu.check_accept(st.accept, res)
        snap = [t.clone() for t in (st.quant.h_full, st.quant.phi, st.pruned.anc_mask, st.accept.path_nodes)]
        if attention != "none":
            snap.append(st.attn_out.clone())
        assert hb.hs_device_error(ctx) == 0     # no device-side wait gave up
        if rep == 1:
            assert all(torch.equal(a, b) for a, b in zip(snap, first))
        first = snap
    return batch, res, st


# ---- small cases: several tiles, a ragged tail, every code path -------------------------------------

SMALL = {
    "c1_small": (synth.CONFIGS["c1_tiny"].scaled(kv_len=(150, 150)), "c1_tiny"),
    "c2_small": (synth.CONFIGS["c2_8b"].scaled(kv_len=(333, 333)), "c2_8b"),
    "c3_small": (synth.CONFIGS["c3_70b"].scaled(kv_len=(200, 200)), "c3_70b"),
    "c4_small": (synth.CONFIGS["c4_ragged"].scaled(batch=5, kv_len=(1, 400)), "c4_ragged"),
    "c5_small": (synth.CONFIGS["c5_long"].scaled(batch=2, kv_len=(700, 700)), "c5_long"),
    # acceptance with deterministic proposals (mode 2), alone and mixed with the two other modes in one batch
    "c3_small_det": (synth.CONFIGS["c3_70b"].scaled(kv_len=(200, 200), accept="deterministic"), "c3_70b"),
    "c4_small_mixed3": (synth.CONFIGS["c4_ragged"].scaled(batch=6, kv_len=(1, 400), accept="mixed3"), "c4_ragged"),
}


@pytest.mark.parametrize("name", sorted(SMALL))
@pytest.mark.parametrize("seed", [11, 12, 13])
def test_small_cases(ctx, name, seed):
    cfg, base = SMALL[name]
    run_and_check(ctx, cfg, pu.policy_for(cfg, base), seed * 100)


# ---- the five configurations at full size -------------------------------------------------------------

def test_c1_tiny_full(ctx):
    cfg = synth.CONFIGS["c1_tiny"]
    run_and_check(ctx, cfg, pu.policy_for(cfg), 1)


def test_c2_8b_full(ctx):
    cfg = synth.CONFIGS["c2_8b"]
    run_and_check(ctx, cfg, pu.policy_for(cfg), 2)


def test_c3_70b_full_systematic_attention(ctx):
    cfg = synth.CONFIGS["c3_70b"]
    run_and_check(ctx, cfg, pu.policy_for(cfg), 3, attention="systematic", attn_pairs=100)


def test_c4_ragged_full_systematic_attention(ctx):
    cfg = synth.CONFIGS["c4_ragged"]
    run_and_check(ctx, cfg, pu.policy_for(cfg), 4, attention="systematic", attn_pairs=8)


def test_c5_long_full_systematic_attention(ctx):
    cfg = synth.CONFIGS["c5_long"]
    run_and_check(ctx, cfg, pu.policy_for(cfg), 5, attention="systematic", attn_pairs=8)


# ---- edge cases -----------------------------------------------------------------------------------------

def test_no_prefix_and_root_only(ctx):
    cfg = synth.CONFIGS["c2_8b"].scaled(kv_len=(0, 0))
    run_and_check(ctx, cfg, pu.policy_for(cfg, "c2_8b"), 7)
    cfg = synth.CONFIGS["c3_70b"].scaled(n_nodes=(1, 1), kv_len=(130, 130))
    run_and_check(ctx, cfg, pu.policy_for(cfg, "c3_70b"), 8)
    cfg = synth.CONFIGS["c4_ragged"].scaled(batch=4, n_nodes=(1, 3), kv_len=(0, 70))
    run_and_check(ctx, cfg, pu.policy_for(cfg, "c4_ragged"), 9)


def test_alternative_readings(ctx):
    """phi_mode / pstar_mode / entropy_mode switches select the other readings of Sec. 4.1."""
    cfg, base = SMALL["c2_small"]
    for mode in (dict(phi_mode=1), dict(pstar_mode=1), dict(entropy_mode=1)):
        pol = dict(pu.policy_for(cfg, base), **mode)
        lo, hi = (0.0, 4.0) if "entropy_mode" in mode else (4.0, 12.0)
        pol["thresholds"] = list(np.linspace(lo, hi, 7))
        run_and_check(ctx, cfg, pol, 300, attention="none")


# ---- one captured graph serves every entropy bin (Sec. 4.3) -----------------------------------------------

@pytest.mark.gpu
def test_graph_replay_across_bins(ctx):
    cfg, base = SMALL["c2_small"]
    policy = pu.policy_for(cfg, base)
    cases = [pu.oracle_case(cfg, policy, seed) for seed in (2100, 2200, 2300, 2400, 2500, 2600)]
    bins = {int(res[0]["pruned"]["bin"]) for _, res in cases}
    assert len(bins) >= 2                      # the seeds land in different regimes (different d', N')
    db = gstep.upload(cases[0][0])
    st = gstep.VerifyStep(ctx, db, policy)
    g = gstep.GraphedStep(st, db)
    for batch, res in cases[1:] + cases[:1]:
        batch = dict(batch, philox_seed=cases[0][0]["philox_seed"], philox_offset=cases[0][0]["philox_offset"])
        gstep.refill(db, batch)
        g.replay()
        torch.cuda.synchronize()
        pu.check_quant(st.quant, batch, res, policy["top_k"])
        pu.check_pruned(st.pruned, res)
        pu.check_attention(st.attn_out, st.attn_lse, batch, res)
        pu.check_accept(st.accept, res)
        assert hb.hs_device_error(ctx) == 0


# ---- a graph per regime, grids sized to the regime's N' (Sec. 4.3, Dynamic Computational Adaptation) ---------------------

def test_regime_graphs_across_bins(ctx):
    cfg, base = SMALL["c2_small"]
    policy = pu.policy_for(cfg, base)
    cases = [pu.oracle_case(cfg, policy, seed) for seed in (2100, 2200, 2300, 2400, 2500, 2600)]
    db = gstep.upload(cases[0][0])
    st = gstep.VerifyStep(ctx, db, policy)
    rs = gstep.RegimeStep(st, db)
    assert rs.bounds == [22, 39, 60]                       # N' of bins 0, 1 and of the rest (62 is capped by the 60 drafted nodes)
    used = set()
    for batch, res in cases[1:] + cases[:1]:
        batch = dict(batch, philox_seed=cases[0][0]["philox_seed"], philox_offset=cases[0][0]["philox_offset"])
        gstep.refill(db, batch)
        rs.replay()
        torch.cuda.synchronize()
        nk = len(res[0]["pruned"]["keep_idx"])
        assert rs.last_bound == min(b for b in rs.bounds if b >= nk)
        used.add(rs.last_bound)
        pu.check_quant(st.quant, batch, res, policy["top_k"])
        pu.check_pruned(st.pruned, res)
        pu.check_attention(st.attn_out, st.attn_lse, batch, res)
        pu.check_accept(st.accept, res)
        assert hb.hs_device_error(ctx) == 0
    assert len(used) >= 2                                  # the seeds land in regimes with different graphs
