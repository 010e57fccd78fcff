"""Oracle: token-tree construction and the integer steps around a verify step.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Paper Section 3.3
("Tree-based Jacobi Decoding", "Retrieval-Augmented Jacobi Decoding"),
Appendix B (token-tree template), Eq. 4 (ahead noise).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np


def validate_tree(parent: Sequence[int]) -> None:
    """A tree is a parent-pointer array in topological order: parent[0] = -1, 0 <= parent[i] < i."""
    if len(parent) == 0 or parent[0] != -1:
        raise ValueError("row 0 must be the root with parent -1")
    for i in range(1, len(parent)):
        if not (0 <= parent[i] < i):
            raise ValueError(f"parent[{i}] = {parent[i]} is not an earlier row")


def depths(parent: Sequence[int]) -> np.ndarray:
    """depth[0] = 0, depth[i] = depth[parent[i]] + 1."""
    validate_tree(parent)
    d = np.zeros(len(parent), np.int32)
    for i in range(1, len(parent)):
        d[i] = d[parent[i]] + 1
    return d


def ancestor_mask(parent: Sequence[int]) -> np.ndarray:
    """mask[i, j] is True iff tree row j is row i itself or one of its ancestors.

    This is the tree part of the sparse attention matrix of token-tree
    verification (Section 2.2, Appendix B): every root-to-leaf path then sees
    exactly what it would see as an ordinary sequence.
    """
    validate_tree(parent)
    m = len(parent)
    mask = np.zeros((m, m), bool)
    for i in range(m):
        j = i
        while j >= 0:
            mask[i, j] = True
            j = parent[j]
    return mask


def pack_mask(mask: np.ndarray) -> np.ndarray:
    """Rows of ``mask`` as little-endian bit words: bit (j % 64) of word j // 64 <=> mask[i, j]."""
    m = mask.shape[0]
    words = (m + 63) // 64
    out = np.zeros((m, words), np.uint64)
    for i in range(m):
        for j in range(m):
            if mask[i, j]:
                out[i, j // 64] |= np.uint64(1) << np.uint64(j % 64)
    return out


def build_tree(root: int, window: Sequence[int],
               branches: Sequence[Sequence[int]]) -> Tuple[np.ndarray, np.ndarray]:
    """Merge the Jacobi window and the retrieved branches into one token tree.

    Row 0 holds ``root``; the window follows as a chain (Section 3.3: every
    path of the tree is an ordinary Jacobi trajectory); each retrieved branch
    is a further chain hanging off the root (Section 3.3: a dedicated
    retrieval path).  Returns (tokens[M], parent[M]).
    """
    tokens: List[int] = [int(root)]
    parent: List[int] = [-1]
    prev = 0
    for t in window:
        tokens.append(int(t))
        parent.append(prev)
        prev = len(tokens) - 1
    for br in branches:
        prev = 0
        for t in br:
            tokens.append(int(t))
            parent.append(prev)
            prev = len(tokens) - 1
    return np.asarray(tokens, np.int32), np.asarray(parent, np.int32)


def ahead_noise(context: Sequence[int], draw: int) -> int:
    """Eq. 4: a noise token is a uniform sample of the tokens ahead of it.

    ``draw`` is a raw non-negative random integer supplied by the caller.
    """
    return int(context[int(draw) % len(context)])


def retrieve(context: Sequence[int], n_branches: int, branch_len: int,
             draws: Sequence[int]) -> List[List[int]]:
    """Prompt-lookup retrieval over all committed tokens (Section 3.3).

    The key is the last g tokens of ``context`` (which ends with the root),
    g = 2 then g = 1.  Scanning backwards, every earlier occurrence of the key
    contributes the tokens that followed it.  The ``n_branches`` most recent
    distinct continuations are kept (g = 2 matches before g = 1 matches).
    Position j of branch r that retrieval cannot fill is ahead noise drawn with
    ``draws[r * branch_len + j]``.
    """
    n = len(context)
    starts: List[int] = []          # index of the first token following a match
    for g in (2, 1):
        if n <= g:
            continue
        key = list(context[n - g:])
        for p in range(n - g - 1, -1, -1):
            if len(starts) >= n_branches:
                break
            if list(context[p:p + g]) == key and (p + g) not in starts:
                starts.append(p + g)
    out: List[List[int]] = []
    for r in range(n_branches):
        br: List[int] = []
        for j in range(branch_len):
            if r < len(starts) and starts[r] + j < n:
                br.append(int(context[starts[r] + j]))
            else:
                br.append(ahead_noise(context, draws[r * branch_len + j]))
        out.append(br)
    return out


def continuation_rows(parent: Sequence[int], best: int) -> List[int]:
    """Rows below ``best`` along its own path: the lowest-index child at every level, down to a leaf."""
    m = len(parent)
    rows: List[int] = []
    cur = best
    while True:
        kids = [c for c in range(cur + 1, m) if parent[c] == cur]
        if not kids:
            return rows
        cur = kids[0]
        rows.append(cur)


def refill_tree(parent: Sequence[int], rank: Sequence[int], node_topk: np.ndarray, best: int,
                context: Sequence[int], draws: Sequence[int], retrieved: Sequence[int]) -> List[int]:
    """Draft tokens of the next step for a static tree template with top-K siblings (Section 3.3, Appendix B).

    The template is ``parent`` plus, for every row i >= 1, ``rank[i]``: rank r >= 0 makes the row the r-th best
    candidate for its position (siblings under one parent carry ranks 0, 1, 2, ...); rank -1 - j makes it slot j of
    the retrieval path(s) and it takes ``retrieved[j]``.  The candidates for depth d come from the d-th row below
    the winner ``best`` along its own path (the chosen path's subsequent predictions): a row of depth d and rank r
    takes ``node_topk[that row][r]``.  Depths the path does not reach are ahead noise over ``context`` (the
    committed tokens, this step's included), row i using ``draws[i - 1]``.  Returns the tokens of rows 1..M-1; row 0
    (the root) is the step's bonus token and is not produced here.  With a chain template and ranks 0 this is
    ``refill_window``.
    """
    depth = depths(parent)
    below = continuation_rows(parent, best)
    out: List[int] = []
    for i in range(1, len(parent)):
        r = int(rank[i])
        if r < 0:
            out.append(int(retrieved[-1 - r]))
        elif depth[i] <= len(below):
            out.append(int(node_topk[below[depth[i] - 1]][r]))
        else:
            out.append(ahead_noise(context, draws[i - 1]))
    return out


def refill_window(parent: Sequence[int], node_pred: Sequence[int], best: int, width: int,
                  context: Sequence[int], draws: Sequence[int]) -> List[int]:
    """Next Jacobi window (Section 3.3): the chosen path's subsequent predictions, then noise.

    Starting below the winning row ``best`` and following the lowest-index
    child at every level, the arg-max at each visited row becomes the next
    guess; the remaining positions are ahead noise over ``context`` (the
    committed tokens including this step's), slot i using ``draws[i]``.
    """
    m = len(parent)
    window: List[int] = []
    cur = best
    while len(window) < width:
        kids = [c for c in range(cur + 1, m) if parent[c] == cur]
        if not kids:
            break
        cur = kids[0]
        window.append(int(node_pred[cur]))
    while len(window) < width:
        window.append(ahead_noise(context, draws[len(window)]))
    return window
