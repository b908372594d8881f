"""Pins of the oracle's tree attention: degenerate closed forms and torch's float64 CPU
scaled_dot_product_attention (causal chain, and an explicit mask for a general tree)."""
import numpy as np
import pytest
import scipy.special
import torch

from oracle import attention, tree


def rand(rng, *shape):
    return rng.standard_normal(shape)


def test_single_key_returns_its_value():
    rng = np.random.default_rng(0)
    q, k, v = rand(rng, 1, 4, 16), rand(rng, 1, 2, 16), rand(rng, 1, 2, 16)
    empty = np.zeros((0, 2, 16))
    out, lse = attention.tree_attention(q, k, v, empty, empty, np.ones((1, 1), bool), 0.25)
    for h in range(4):
        assert np.allclose(out[0, h], v[0, h // 2], atol=1e-14)
        assert lse[0, h] == pytest.approx(0.25 * q[0, h] @ k[0, h // 2], rel=1e-12)


def test_equal_keys_give_mean_value():
    rng = np.random.default_rng(1)
    L, n = 9, 3
    key = rand(rng, 1, 1, 8)
    kc, kt = np.repeat(key, L, 0), np.repeat(key, n, 0)
    vc, vt = rand(rng, L, 1, 8), rand(rng, n, 1, 8)
    mask = np.tril(np.ones((n, n), bool))
    out, lse = attention.tree_attention(rand(rng, n, 2, 8), kt, vt, kc, vc, mask, 0.3)
    for i in range(n):
        want = np.concatenate([vc[:, 0], vt[: i + 1, 0]]).mean(0)
        assert np.allclose(out[i, 0], want, atol=1e-13) and np.allclose(out[i, 1], want, atol=1e-13)


def test_chain_without_prefix_is_causal_attention():
    rng = np.random.default_rng(2)
    n, hq, hkv, D = 11, 4, 2, 16
    q, k, v = rand(rng, n, hq, D), rand(rng, n, hkv, D), rand(rng, n, hkv, D)
    mask = np.tril(np.ones((n, n), bool))
    empty = np.zeros((0, hkv, D))
    out, _ = attention.tree_attention(q, k, v, empty, empty, mask, D ** -0.5)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(hq // hkv, 0)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(hq // hkv, 0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    assert np.allclose(out, ref[0].permute(1, 0, 2).numpy(), atol=1e-12)


@pytest.mark.parametrize("seed", range(3))
def test_tree_with_prefix_against_sdpa(seed):
    rng = np.random.default_rng(10 + seed)
    n, L, hq, hkv, D = 14, 37, 6, 2, 8
    parent = np.array([-1] + [int(rng.integers(0, i)) for i in range(1, n)])
    S = -np.arange(n, dtype=float)
    mask = tree.prune(parent, S, 99, 99)["mask"]
    q, kt, vt = rand(rng, n, hq, D), rand(rng, n, hkv, D), rand(rng, n, hkv, D)
    kc, vc = rand(rng, L, hkv, D), rand(rng, L, hkv, D)
    out, lse = attention.tree_attention(q, kt, vt, kc, vc, mask, D ** -0.5)
    g = hq // hkv
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(np.concatenate([kc, kt])).permute(1, 0, 2).repeat_interleave(g, 0)[None]
    tv = torch.from_numpy(np.concatenate([vc, vt])).permute(1, 0, 2).repeat_interleave(g, 0)[None]
    full = torch.from_numpy(np.concatenate([np.ones((n, L), bool), mask], 1))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=full)
    assert np.allclose(out, ref[0].permute(1, 0, 2).numpy(), atol=1e-12)
    # normaliser against scipy's logsumexp on hand-built scores
    i, h = n - 1, 3
    keys = np.concatenate([kc[:, h // g], kt[:, h // g]])
    s = (keys @ q[i, h]) * D ** -0.5
    vis = np.concatenate([np.ones(L, bool), mask[i]])
    assert lse[i, h] == pytest.approx(scipy.special.logsumexp(s[vis]), rel=1e-12)


def test_sampled_rows_match_full():
    rng = np.random.default_rng(5)
    n, L = 5, 6
    args = (rand(rng, n, 2, 4), rand(rng, n, 1, 4), rand(rng, n, 1, 4), rand(rng, L, 1, 4),
            rand(rng, L, 1, 4), np.tril(np.ones((n, n), bool)), 0.5)
    full, _ = attention.tree_attention(*args)
    part, _ = attention.tree_attention(*args, rows=[(3, 1)])
    assert np.array_equal(part[3, 1], full[3, 1]) and np.isnan(part[0, 0]).all()
