"""GPU parity of the stratifier training (Sec. 4.2, Eq. 2): the thresholds fitted on the device equal the CPU
oracle's, on synthetic (entropy, rank) pairs and on pairs the verification path itself emits (phi_star of
hs_entropy_quantify, terminal_rank of hs_accept_path); App. A.4's Jaccard comparison across depths runs on them."""
import time

import numpy as np
import pytest
import torch

from oracle import cart as ocart
from paper_2505_13254_b200 import binding as hb
from paper_2505_13254_b200 import step as gstep
from paper_2505_13254_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu


def clear_margin(x, y, depth, rel=1e-7):
    """True if, in every node of the oracle's tree, the best split beats the runner-up by a clear margin (the
    device scores splits from running sums, the oracle from the definition: near-ties may fall either way)."""
    x, y = np.asarray(x, dtype=np.float64), np.asarray(y, dtype=np.float64)
    nodes = [(-np.inf, np.inf)]
    for _ in range(depth):
        nxt = []
        for lo, hi in nodes:
            sel = (x >= lo) & (x < hi)
            xs = np.unique(x[sel])
            losses = sorted(ocart.split_loss(x[sel], y[sel], 0.5 * (a + b)) for a, b in zip(xs[:-1], xs[1:]))
            if len(losses) > 1 and losses[1] - losses[0] <= rel * max(1.0, losses[0]):
                return False
            if len(xs) < 2:
                return False                                  # (a node that cannot be split: draw again)
            s = ocart.best_split(x[sel], y[sel])[0]
            nxt += [(lo, s), (s, hi)]
        nodes = nxt
    return True


@pytest.mark.parametrize("n,depth", [(600, 3), (3000, 3), (1500, 5), (700, 6), (2049, 2)])
def test_thresholds_match_the_oracle_on_synthetic_pairs(n, depth):
    ctx = hb.Context(0, hb.hs_cart_workspace_bytes(1 << 20) + (1 << 20))
    seed = 0
    while True:
        rng = np.random.default_rng(1000 * n + seed)
        x = rng.gamma(4.0, 2.0, n).astype(np.float32)                         # entropies: positive, skewed
        y = np.clip(np.round(0.4 * x ** 1.5 + rng.normal(0, 3, n)), 0, 59).astype(np.float32)   # ranks 0 .. 59
        if n > 100:
            x[rng.integers(0, n, n // 10)] = x[rng.integers(0, n, n // 10)]   # repeated feature values
        if clear_margin(x, y, depth):
            break
        seed += 1
    want = ocart.fit_thresholds(x, y, depth)
    th, status = hb.hs_cart_fit(ctx, torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda(), depth)
    torch.cuda.synchronize()
    assert int(status) == 0
    assert np.allclose(th.cpu().numpy().astype(np.float64), want, rtol=1e-6, atol=1e-6)
    assert hb.hs_device_error(ctx) == 0
    ctx.close()


def test_a_node_with_one_feature_value_is_reported():
    ctx = hb.Context(0, 8 << 20)
    x = torch.ones(64, device="cuda")
    y = torch.arange(64, device="cuda", dtype=torch.float32)
    th, status = hb.hs_cart_fit(ctx, x, y, 3)
    torch.cuda.synchronize()
    assert int(status) == hb.HS_ERR_SHAPE and torch.isnan(th).all()
    with pytest.raises(hb.HsError):
        hb.hs_cart_fit(ctx, x[:4], y[:4], 3)                     # fewer samples than leaves
    ctx.close()


def test_training_on_pairs_from_the_verification_path():
    """(Phi(P*), Terminal Confidence Rank) pairs from 96 synthetic trees verified on the device train the
    stratifier; the thresholds equal the oracle's on the same pairs, become the policy of the next step, and the
    low-entropy sets of deeper trees are compared with the 3-layer one (App. A.4)."""
    cfg = synth.CONFIGS["c1_tiny"].scaled(batch=32, vocab=4096, kv_len=(8, 8), n_nodes=(30, 60))
    policy = pu.policy_for(cfg, "c1_tiny")
    ctx = hb.Context(0, 64 << 20)
    xs, ys = [], []
    for seed in (7001, 7002, 7003):
        db = gstep.upload(synth.make_batch(cfg, seed, with_attention=False))
        st = gstep.VerifyStep(ctx, db, policy)
        st.quantify(db); st.prune(db); st.accept_path(db)
        xs.append(st.quant.phi_star.clone()); ys.append(st.accept.terminal_rank.float())
    x, y = torch.cat(xs), torch.cat(ys)
    th, status = hb.hs_cart_fit(ctx, x, y, 3)
    torch.cuda.synchronize()
    assert int(status) == 0
    xh, yh = x.cpu().numpy(), y.cpu().numpy()
    if clear_margin(xh, yh, 3):
        assert np.allclose(th.cpu().numpy(), ocart.fit_thresholds(xh, yh, 3), rtol=1e-6, atol=1e-6)
    assert all(a < b for a, b in zip(th.tolist()[:-1], th.tolist()[1:]))
    # the trained thresholds drive the next step
    policy2 = dict(policy, thresholds=th.tolist())
    db = gstep.upload(synth.make_batch(cfg, 7004, with_attention=False))
    st = gstep.VerifyStep(ctx, db, policy2)
    st.quantify(db); st.prune(db)
    torch.cuda.synchronize()
    assert np.array_equal(st.pruned.bin.cpu().numpy(), ocart.bins_of(st.quant.phi_star.cpu().numpy(), th.cpu().numpy()))
    # App. A.4: the low-entropy set of the 3-layer tree against deeper trees
    low3 = ocart.low_entropy_set(xh, th.cpu().numpy())
    for d in (4, 5):
        thd, sd = hb.hs_cart_fit(ctx, x, y, d)
        if int(sd) == 0:
            j = ocart.jaccard(low3, ocart.low_entropy_set(xh, thd.cpu().numpy()))
            assert 0.0 <= j <= 1.0
            print(f"Jaccard(3 layers, {d} layers) = {j:.2f} on {len(xh)} synthetic trees")
    ctx.close()


def test_a_million_pairs_train_in_well_under_a_second():
    n = 1 << 20
    ctx = hb.Context(0, hb.hs_cart_workspace_bytes(n) + (1 << 20))
    g = torch.Generator(device="cuda").manual_seed(1)
    x = torch.rand(n, device="cuda", generator=g) * 12
    y = torch.clamp(torch.round(x * 4 + torch.randn(n, device="cuda", generator=g) * 5), 0, 59)
    hb.hs_cart_fit(ctx, x, y, 3)
    torch.cuda.synchronize()
    t = time.perf_counter()
    th, status = hb.hs_cart_fit(ctx, x, y, 3)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t
    assert int(status) == 0 and all(a < b for a, b in zip(th.tolist()[:-1], th.tolist()[1:]))
    print(f"hs_cart_fit on {n} pairs: {dt * 1e3:.1f} ms (the paper reports under 3 s for its CPU training)")
    assert dt < 1.0
    ctx.close()
