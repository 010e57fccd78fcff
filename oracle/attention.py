"""Oracle: tree-masked attention by its definition.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Token-tree verification
(paper Section 2.2 and Appendix B): several candidate continuations are scored
in one forward by masking attention so that each tree row sees the cached
prefix and its own ancestors.
"""
from __future__ import annotations

import numpy as np

from .tree import ancestor_mask


def tree_attention(q: np.ndarray, k_prefix: np.ndarray, v_prefix: np.ndarray,
                   k_tree: np.ndarray, v_tree: np.ndarray, parent) -> np.ndarray:
    """out[i, h] = sum_j softmax_j(q[i,h] . k[h,j] / sqrt(D)) v[h,j] over the visible set of row i.

    q: [M, H, D]; k_prefix, v_prefix: [Hkv, S, D] (S may be 0); k_tree, v_tree:
    [Hkv, M, D]; parent: [M].  The visible set of row i is all S prefix rows plus
    the tree rows j with ``ancestor_mask(parent)[i, j]``.  With grouped-query
    attention (Hkv < H, H a multiple of Hkv) query head h reads K/V head
    h // (H // Hkv); Hkv = H is ordinary multi-head attention.  Returns [M, H, D] fp64.
    """
    q = np.asarray(q, np.float64)
    kp, vp = np.asarray(k_prefix, np.float64), np.asarray(v_prefix, np.float64)
    kt, vt = np.asarray(k_tree, np.float64), np.asarray(v_tree, np.float64)
    m, n_heads, d = q.shape
    mask = ancestor_mask(parent)
    out = np.zeros((m, n_heads, d), np.float64)
    scale = 1.0 / np.sqrt(float(d))
    group = n_heads // kp.shape[0]
    for h in range(n_heads):
        g = h // group
        for i in range(m):
            vis = np.nonzero(mask[i])[0]
            keys = np.concatenate([kp[g], kt[g][vis]], axis=0)
            vals = np.concatenate([vp[g], vt[g][vis]], axis=0)
            s = (keys @ q[i, h]) * scale
            p = np.exp(s - s.max())
            p /= p.sum()
            out[i, h] = p @ vals
    return out
