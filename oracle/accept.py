"""Oracle: per-node arg-max, greedy longest-path acceptance, KV compaction.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Paper Eq. 1 (greedy
target), Section 3.3 (the longest accepted path is chosen; candidate
generation and verification happen in the same forward, so the prediction of
every row is an output).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

from .tree import depths


def node_argmax(logits: np.ndarray) -> np.ndarray:
    """Greedy prediction of every row (Eq. 1); equal logits resolve to the smallest token id."""
    logits = np.asarray(logits, np.float64)
    out = np.zeros(logits.shape[0], np.int32)
    for i in range(logits.shape[0]):
        out[i] = int(np.argmax(logits[i]))        # numpy returns the first maximiser
    return out


def node_topk(logits: np.ndarray, k: int) -> np.ndarray:
    """The k most likely token ids of every row, best first (Appendix B: the tree holds the top-K candidates of a
    draft position as siblings).  Order: larger logit first, equal logits by ascending token id; column 0 is
    ``node_argmax``.  Returns [M, k] int32."""
    logits = np.asarray(logits, np.float64)
    out = np.zeros((logits.shape[0], k), np.int32)
    for i in range(logits.shape[0]):
        order = sorted(range(logits.shape[1]), key=lambda v: (-logits[i, v], v))
        out[i] = order[:k]
    return out


def top2_margin(logits: np.ndarray) -> np.ndarray:
    """Gap between the largest and second-largest logit of every row (0 for an exact tie)."""
    logits = np.asarray(logits, np.float64)
    part = np.partition(logits, logits.shape[1] - 2, axis=1)
    return part[:, -1] - part[:, -2]


def accept_path(tokens: Sequence[int], parent: Sequence[int],
                node_pred: Sequence[int]) -> Tuple[int, List[int], int]:
    """Greedy acceptance over the tree (Section 3.3).

    ok[0] = True; ok[i] = ok[parent[i]] and tokens[i] == node_pred[parent[i]].
    The winner is the accepted row of largest depth, smallest row index among
    equals.  Returns (k, path, bonus): k = depth of the winner, path = rows
    from the root to the winner (k + 1 entries), bonus = node_pred[winner].
    """
    depth = depths(parent)
    m = len(parent)
    ok = [False] * m
    ok[0] = True
    for i in range(1, m):
        ok[i] = ok[parent[i]] and int(tokens[i]) == int(node_pred[parent[i]])
    best = 0
    for i in range(1, m):
        if ok[i] and depth[i] > depth[best]:
            best = i
    path: List[int] = []
    j = best
    while j >= 0:
        path.append(j)
        j = int(parent[j])
    path.reverse()
    return int(depth[best]), path, int(node_pred[best])


def compact_rows(cache: np.ndarray, seq_len: int, path: Sequence[int]) -> int:
    """Keep the accepted rows contiguous after the prefix.

    ``cache`` is [..., rows, D] with the tree's rows stored at seq_len + row.
    Row path[j] moves to seq_len + j for j = 0..k (path[0] = 0 is the root and
    stays).  Returns the new length seq_len + k + 1.
    """
    src = [seq_len + int(r) for r in path]
    kept = cache[..., src, :].copy()
    cache[..., seq_len:seq_len + len(path), :] = kept
    return seq_len + len(path)
