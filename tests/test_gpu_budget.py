"""GPU parity of Top-N reranking under a token budget (App. A.8 reading): hs_stratify_prune_budget against the
oracle's reallocation followed by the oracle's pruning with the reallocated counts."""
import numpy as np
import pytest
import torch

from oracle import budget as obudget
from oracle import tree as otree
from paper_2505_13254_b200 import binding as hb
from paper_2505_13254_b200 import step as gstep
from paper_2505_13254_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu

CFG = synth.CONFIGS["c4_ragged"].scaled(batch=8, vocab=8192, n_nodes=(12, 60), kv_len=(1, 40))


@pytest.fixture(scope="module")
def case():
    policy = pu.policy_for(CFG, "c4_ragged")
    policy["thresholds"] = [float(t) for t in np.linspace(2.0, 12.0, 7)]       # (small vocabulary: other entropies)
    batch, res = pu.oracle_case(CFG, policy, 5100, attention="none")
    return policy, batch, res


def expected(policy, batch, res, slo, budget):
    n_prime = [r["pruned"]["n_prime"] for r in res]
    d_prime = [r["pruned"]["d_prime"] for r in res]
    elig = [int((r["scores"]["depth"] <= d_prime[b]).sum()) for b, r in enumerate(res)]
    n_final = obudget.reallocate(n_prime, elig, slo, budget)
    out, margin = [], np.inf
    for b, r in enumerate(res):
        lo, hi = batch["node_off"][b], batch["node_off"][b + 1]
        S = r["scores"]["S"]
        pr = otree.prune(batch["parent"][lo:hi], S, d_prime[b], n_final[b])
        pr.update(bin=r["pruned"]["bin"], d_prime=d_prime[b], n_prime=n_prime[b])
        out.append(dict(pruned=pr))
        order = sorted((i for i in range(len(S)) if r["scores"]["depth"][i] <= d_prime[b]), key=lambda i: (-S[i], i))
        if 0 < n_final[b] < len(order):
            margin = min(margin, S[order[n_final[b] - 1]] - S[order[n_final[b]]])
    return out, n_final, margin


@pytest.mark.parametrize("kind", ["generous", "tight", "exact", "starved", "huge"])
def test_budgeted_pruning_matches_the_oracle(case, kind):
    policy, batch, res = case
    ctx = hb.Context(0, 64 << 20)
    B = CFG.batch
    rng = np.random.default_rng(len(kind))
    slo = rng.integers(0, 3, B).tolist()
    base = sum(min(r["pruned"]["n_prime"], int((r["scores"]["depth"] <= r["pruned"]["d_prime"]).sum())) for r in res)
    budgets = {"generous": [base + 37, base + 90, base + 5], "tight": [base - 41, base - 13, base - 77],
               "exact": [base], "starved": [3], "huge": [100000]}[kind]
    for budget in budgets:
        want, n_final, margin = expected(policy, batch, res, slo, budget)
        if margin <= 1e-4:
            continue                                     # a cut through a near-tie of path confidences: skip this budget
        db = gstep.upload(batch)
        st = gstep.VerifyStep(ctx, db, policy)
        st.quantify(db)
        hb.hs_stratify_prune_budget(ctx, db.tree, st.quant, policy, torch.tensor(slo, dtype=torch.int32, device="cuda"),
                                    budget, out=st.pruned)
        torch.cuda.synchronize()
        assert st.pruned.n_keep.tolist() == n_final
        assert sum(n_final) <= max(budget, B)
        pu.check_pruned(st.pruned, want)
        # the reallocated tree is a valid input of the rest of the step
        st.accept_path(db)
        torch.cuda.synchronize()
        assert st.accept.status.tolist() == [0] * B
        assert hb.hs_device_error(ctx) == 0
    ctx.close()


def test_without_pressure_the_budget_changes_nothing_when_trees_are_small(case):
    """A budget that covers every eligible node keeps every eligible node."""
    policy, batch, res = case
    ctx = hb.Context(0, 64 << 20)
    db = gstep.upload(batch)
    st = gstep.VerifyStep(ctx, db, policy)
    st.quantify(db)
    hb.hs_stratify_prune_budget(ctx, db.tree, st.quant, policy, torch.zeros(CFG.batch, dtype=torch.int32, device="cuda"),
                                1 << 20, out=st.pruned)
    torch.cuda.synchronize()
    elig = [int((r["scores"]["depth"] <= r["pruned"]["d_prime"]).sum()) for r in res]
    assert st.pruned.n_keep.tolist() == elig
    ctx.close()
