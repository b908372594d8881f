"""CPU oracle for the HeteroSpec draft-tree verification step (arXiv 2505.13254).

TEST INFRASTRUCTURE ONLY.  A plain, slow, float64 numpy restatement of what each
step of the verification path computes, written from the paper's definitions.
It shares no code with the CUDA path and must never be imported by it; only the
tests, the smoke check and the benchmark's CPU-baseline leg call it.

Steps (one module each):
  row_stats   Eq. 1 inner sum: softmax, Shannon entropy, Top-K and its entropies
  tree        path aggregation Phi / V_i, operational path P*, entropy bins,
              d' and N' policy (Sec. 4.2-4.3), Top-N' pruning and the tree mask
  attention   tree-masked attention of kept nodes over prefix + tree (Sec. 2.2)
  accept      greedy and rejection-sampling acceptance (Sec. 2.1)
  philox      Philox4x32-10 uniforms (Salmon et al., SC'11), own implementation
  expand      draft-tree expansion and reranking (Sec. 2.2), the step ahead of verification

Parity pins: every function is pinned by tests/test_oracle_*.py against closed
forms, invariants, brute force or a published known answer, except the numeric
values of the seven entropy thresholds, which the paper does not publish
("parity unpinned": thresholds are an input here).
"""

from . import accept, attention, expand, philox, row_stats, step, tree  # noqa: F401


def bf16_bits_to_f64(bits):
    """Widen bfloat16 bit patterns (uint16) to float64 exactly."""
    import numpy as np
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
