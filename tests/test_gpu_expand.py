"""GPU parity of the draft-tree expansion and reranking (Sec. 2.2; Sec. 4.3 for the number of levels and N'):
the device grows the candidate tree level by level from the Top-K statistics that hs_entropy_quantify writes for
the frontier rows, and the result must equal the CPU oracle's tree candidate by candidate; the reranked tree must
equal the oracle's and feed the verification calls."""
import numpy as np
import pytest
import torch

from oracle import expand as oexp
from paper_2505_13254_b200 import binding as hb
from paper_2505_13254_b200 import synth

pytestmark = pytest.mark.gpu


def toy_model(vocab, seed, b):
    """A deterministic stand-in for the draft model: logits after a token path, bf16-exact values."""
    def row(path):
        r = np.random.default_rng([seed, b, len(path)] + list(path))
        x = r.standard_normal(vocab).astype(np.float32) * np.float32(2.5)
        return synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x))
    return row


def margins(cand, k, n_tops):
    """Smallest value gap at a frontier cut or a reranking cut (the device decides these in fp32)."""
    S, dep = cand["S"], cand["depth"]
    m = np.inf
    for level in range(1, int(dep.max()) + 1):
        s = np.sort(S[dep == level])[::-1]
        if len(s) > k:
            m = min(m, s[k - 1] - s[k])
    s = np.sort(S)[::-1]
    for n in n_tops:
        if n < len(s):
            m = min(m, s[n - 1] - s[n])
    return m


@pytest.mark.parametrize("k,depth,vocab,batch", [(10, 8, 32000, 2), (4, 12, 5000, 3), (16, 3, 128256, 1), (2, 5, 64, 4)])
def test_expansion_and_reranking_match_the_oracle(k, depth, vocab, batch):
    ctx = hb.Context(0, 64 << 20)
    dev = torch.device("cuda:0")
    n_tops = [60, 22, 39][:batch] + [7] * max(0, batch - 3)
    seed = 0
    while True:                                           # a draw without near-ties at the cuts
        models = [toy_model(vocab, 1000 + seed, b) for b in range(batch)]
        cands = [oexp.expand(lambda c, path, m=models[b]: m(path), depth, k) for b in range(batch)]
        if min(margins(c, k, [n_tops[b]]) for b, c in enumerate(cands)) > 1e-4:
            break
        seed += 1
    cap = 1 + k + (depth - 1) * k * k
    st = hb.ExpandState(batch, cap, k, dev)
    hb.hs_expand_init(ctx, st)
    # a dummy star tree of k nodes per sequence carries the k frontier rows through hs_entropy_quantify
    i32 = lambda a: torch.tensor(a, dtype=torch.int32, device=dev)
    tree = hb.TreeBatch(i32([b * k for b in range(batch + 1)]), i32(([-1] + [0] * (k - 1)) * batch), i32([0] * (k * batch)),
                        batch, k * batch)
    policy = dict(thresholds=list(np.linspace(1, 7, 7)), d_base=depth, alpha=(depth + 1) // 2, n_default=60, top_k=k,
                  gamma_pct=[30, 60, 100], phi_mode=0, pstar_mode=0, entropy_mode=0)
    paths = [[[]] for _ in range(batch)]                  # token path of every candidate, from the oracle's tree
    for b, c in enumerate(cands):
        for cid in range(1, len(c["S"])):
            paths[b].append(paths[b][int(c["parent"][cid])] + [int(c["token"][cid])])
    for level in range(depth):
        rows = np.zeros((batch * k, vocab), dtype=np.float32)
        for b, c in enumerate(cands):
            fr = c["frontiers"][level]
            got = st.frontier[b, : int(st.n_frontier[b])].tolist()
            assert got == fr, (level, b, got, fr)             # the device chose the same nodes to expand
            for j, cid in enumerate(fr):
                rows[b * k + j] = models[b](paths[b][cid])
        logits = torch.from_numpy(synth.f32_to_bf16_bits(rows).view(np.int16)).to(dev).view(torch.bfloat16)
        q = hb.hs_entropy_quantify(ctx, tree, logits, policy)
        hb.hs_expand_level(ctx, st, q)
    torch.cuda.synchronize()
    assert st.status.tolist() == [0] * batch
    for b, c in enumerate(cands):
        n = len(c["S"])
        assert int(st.n_cand[b]) == n == cap
        assert np.array_equal(st.parent[b, :n].cpu().numpy(), c["parent"])
        assert np.array_equal(st.token[b, 1:n].cpu().numpy(), c["token"][1:])
        assert np.array_equal(st.depth[b, :n].cpu().numpy(), c["depth"])
        assert np.allclose(st.logc[b, :n].cpu().numpy(), c["logc"], rtol=1e-4, atol=1e-5)
        assert np.allclose(st.score[b, :n].cpu().numpy(), c["S"], rtol=1e-4, atol=1e-5)
    # reranking with a Top-N per sequence (as Sec. 4.3 gives every sequence its own N')
    node_off, parent, token, cand_id, tdepth = hb.hs_rerank(ctx, st, i32(n_tops[:batch]), 60)
    torch.cuda.synchronize()
    off = node_off.tolist()
    for b, c in enumerate(cands):
        want = oexp.rerank(c, n_tops[b])
        sl = slice(off[b], off[b + 1])
        assert off[b + 1] - off[b] == len(want["cand_id"])
        assert np.array_equal(cand_id[sl].cpu().numpy(), want["cand_id"])
        assert np.array_equal(parent[sl].cpu().numpy(), want["parent"])
        assert np.array_equal(token[sl].cpu().numpy()[1:], want["token"][1:])
        assert np.array_equal(tdepth[sl].cpu().numpy(), want["depth"])
    # one more level than the arrays hold is refused per sequence, not by a fault
    hb.hs_expand_level(ctx, st, q)
    torch.cuda.synchronize()
    assert st.status.tolist() == [hb.HS_ERR_SHAPE] * batch
    assert hb.hs_device_error(ctx) == 0
    ctx.close()
