"""Oracle step 5: tree-masked attention (test infrastructure only).

The target model scores every kept draft token in one pass (Sec. 2.2): kept
node i attends to the whole accepted prefix and, inside the tree, only to itself
and its ancestors.  Plain float64 softmax attention, one (node, head) at a time.
"""

import numpy as np


def tree_attention(q, k_tree, v_tree, k_cache, v_cache, mask, scale, rows=None):
    """q [n, Hq, D]; k_tree, v_tree [n, Hkv, D]; k_cache, v_cache [L, Hkv, D]; mask [n, n] bool.

    Query head h uses key/value head h // (Hq // Hkv).  Returns (out [n, Hq, D], lse [n, Hq]);
    lse is the natural-log normaliser of the scaled scores.  ``rows`` restricts the computation
    to some (node, head) pairs, the other entries are left NaN (for sampled checks at full size).
    """
    q = np.asarray(q, dtype=np.float64)
    n, hq, D = q.shape
    hkv = k_tree.shape[1]
    g = hq // hkv
    L = k_cache.shape[0]
    out = np.full((n, hq, D), np.nan)
    lse = np.full((n, hq), np.nan)
    pairs = rows if rows is not None else [(i, h) for i in range(n) for h in range(hq)]
    for i, h in pairs:
        kh = h // g
        keys = np.concatenate([np.asarray(k_cache[:, kh], dtype=np.float64),
                               np.asarray(k_tree[:, kh], dtype=np.float64)])
        vals = np.concatenate([np.asarray(v_cache[:, kh], dtype=np.float64),
                               np.asarray(v_tree[:, kh], dtype=np.float64)])
        visible = np.concatenate([np.ones(L, dtype=bool), np.asarray(mask[i], dtype=bool)])
        s = (keys @ q[i, h]) * scale
        s = s[visible]
        m = s.max()
        e = np.exp(s - m)
        z = e.sum()
        out[i, h] = (e / z) @ vals[visible]
        lse[i, h] = m + np.log(z)
    return out, lse
