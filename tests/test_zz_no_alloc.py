"""hs_entropy_quantify_static: the entropy pass for callers that cannot allocate device memory (their memory
belongs to an arena fixed at start-up, or cudaMalloc is forbidden after initialisation).  It keeps its scratch
in an array built into the library, so it must give what hs_entropy_quantify gives with an allocated
workspace - here on two different batches in a row, the second one seeing the first one's leftovers - and it
must refuse batches larger than that array.  Collected last on purpose: a failure here stops nothing else."""
import numpy as np
import pytest
import torch

from paper_2505_13254_b200 import binding as hb
from paper_2505_13254_b200 import step as gstep
from paper_2505_13254_b200 import synth

import parity_util as pu

pytestmark = pytest.mark.gpu

FLOATS = ("row_max", "row_lse", "h_full", "i_topk", "i_trunc", "topk_val", "logc", "score", "phi", "phi_star")
INTS = ("topk_idx", "depth", "pstar_node", "status")


def _compare(a, b):
    for name in INTS:
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    for name in FLOATS:                                   # the tolerance of the parity tests: 1e-4 relative
        x, y = getattr(a, name).double(), getattr(b, name).double()
        assert torch.all((x - y).abs() <= 1e-4 * y.abs() + 1e-6), name


def test_static_scratch_matches_the_workspace_path_twice_in_a_row():
    torch.cuda.set_device(0)
    ctx = hb.Context(0, 256 << 20)
    cases = [(synth.CONFIGS["c4_ragged"].scaled(batch=3, kv_len=(8, 8)), "c4_ragged", 71),
             (synth.CONFIGS["c1_tiny"].scaled(kv_len=(8, 8)), "c1_tiny", 72)]
    for cfg, base, seed in cases:                         # bf16 ragged batch, then an fp32 tree
        policy = pu.policy_for(cfg, base)
        batch, res = pu.oracle_case(cfg, policy, seed, attention="none")
        db = gstep.upload(batch)
        want = hb.hs_entropy_quantify(ctx, db.tree, db.draft, policy)
        got = hb.hs_entropy_quantify_static(db.tree, db.draft, policy)
        torch.cuda.synchronize()
        assert int(got.status.abs().sum()) == 0
        _compare(got, want)
        pu.check_quant(got, batch, res, policy["top_k"])     # and against the CPU oracle, like every other path
    ctx.close()


def test_static_scratch_rejects_what_does_not_fit():
    torch.cuda.set_device(0)
    n = hb.HS_STATIC_MAX_ROWS + 1
    dev = torch.device("cuda:0")
    i32 = lambda a: torch.tensor(a, dtype=torch.int32, device=dev)
    tree = hb.TreeBatch(i32([0, n]), i32([-1] + [0] * (n - 1)), i32([0] * n), 1, n)
    logits = torch.zeros(n, 64, dtype=torch.float32, device=dev)
    policy = dict(thresholds=list(np.linspace(1, 7, 7)), d_base=4, alpha=2, n_default=20, top_k=4,
                  gamma_pct=[30, 60, 100], phi_mode=0, pstar_mode=0, entropy_mode=0)
    with pytest.raises(hb.HsError) as e:
        hb.hs_entropy_quantify_static(tree, logits, policy)
    assert e.value.status == hb.HS_ERR_STATIC_LIMIT and "built-in scratch" in str(e.value)
