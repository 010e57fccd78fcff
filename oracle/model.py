"""Oracle: LLaMA-family decoder forward over tree rows, greedy decoding drivers.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Paper Eq. 1 (the
autoregressive greedy target), Section 2.1 (Jacobi decoding), Section 3.3
(TR-Jacobi: one forward verifies the tree and produces the next candidates).
"""
from __future__ import annotations

from typing import Callable, Dict, List, Sequence

import numpy as np

from .accept import accept_path, compact_rows, node_argmax, node_topk
from .attention import tree_attention
from .tree import build_tree, depths, refill_tree, refill_window, retrieve, ahead_noise


def rmsnorm(h: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain along the last axis."""
    ms = np.mean(h * h, axis=-1, keepdims=True)
    return h / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, half-split pairing: (x[i], x[i + D/2]) is rotated by pos * theta^(-2i/D).

    x: [M, H, D]; pos: [M].
    """
    d = x.shape[-1]
    half = d // 2
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = np.asarray(pos, np.float64)[:, None] * inv_freq[None, :]        # [M, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def store_bf16(x: np.ndarray) -> np.ndarray:
    """Value a bf16 tensor holds after ``x`` is stored in it: nearest bf16, ties to even (as fp64)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.float64)


class KVCache:
    """K and V of every layer, [L, Hkv, capacity, D] fp64, and the number of committed rows."""

    def __init__(self, n_layers: int, n_heads: int, capacity: int, head_dim: int):
        self.k = np.zeros((n_layers, n_heads, capacity, head_dim), np.float64)
        self.v = np.zeros((n_layers, n_heads, capacity, head_dim), np.float64)
        self.seq_len = 0


class Decoder:
    """Random-init LLaMA-shaped decoder.

    ``layers`` is indexable by layer and yields the dict produced by the input
    generator (``attn_norm``, ``wqkv``, ``wo``, ``mlp_norm``, ``w_gate_up``,
    ``w_down``; matrices are [d_out, d_in]); ``glob`` holds ``embed``,
    ``lm_head``, ``final_norm``.
    """

    def __init__(self, cfg, layers, glob: Dict[str, np.ndarray]):
        self.cfg = cfg
        self.layers = layers
        self.glob = glob

    def new_cache(self, capacity: int) -> KVCache:
        c = self.cfg
        return KVCache(c.n_layers, getattr(c, "kv_heads", c.n_heads), capacity, c.head_dim)

    def forward_rows(self, cache: KVCache, tokens: Sequence[int], parent: Sequence[int]) -> np.ndarray:
        """Logits [M, V] of the M tree rows given the cache's first ``seq_len`` rows.

        K/V of tree row i is stored at cache row seq_len + i; ``seq_len`` itself
        is left unchanged (the caller commits rows by compaction).
        """
        c = self.cfg
        m, s = len(tokens), cache.seq_len
        n_heads, hd = c.n_heads, c.head_dim
        kv_heads = getattr(c, "kv_heads", n_heads)          # grouped-query attention when smaller than n_heads
        pos = s + depths(parent)
        # bf16 configs: q and the K/V cache rows are bf16 tensors (the cache is stored in bf16 by the
        # config's definition and q is the other operand of the attention op); what such a tensor holds
        # is the rounded value.  Everything else, and all arithmetic, stays fp64.
        store = store_bf16 if c.dtype == "bf16" else (lambda t: t)
        h = np.asarray(self.glob["embed"], np.float64)[np.asarray(tokens, np.int64)]
        for l in range(c.n_layers):
            w = self.layers[l]
            x = rmsnorm(h, np.asarray(w["attn_norm"], np.float64), c.rms_eps)
            qkv = x @ np.asarray(w["wqkv"], np.float64).T
            nq, nkv = n_heads * hd, kv_heads * hd
            q = qkv[:, :nq].reshape(m, n_heads, hd)
            k = qkv[:, nq:nq + nkv].reshape(m, kv_heads, hd)
            v = qkv[:, nq + nkv:].reshape(m, kv_heads, hd)
            q, k, v = store(rope(q, pos, c.rope_theta)), store(rope(k, pos, c.rope_theta)), store(v)
            cache.k[l][:, s:s + m, :] = k.transpose(1, 0, 2)
            cache.v[l][:, s:s + m, :] = v.transpose(1, 0, 2)
            att = tree_attention(q, cache.k[l][:, :s], cache.v[l][:, :s],
                                 cache.k[l][:, s:s + m], cache.v[l][:, s:s + m], parent)
            h = h + att.reshape(m, n_heads * hd) @ np.asarray(w["wo"], np.float64).T
            x = rmsnorm(h, np.asarray(w["mlp_norm"], np.float64), c.rms_eps)
            gu = x @ np.asarray(w["w_gate_up"], np.float64).T
            act = silu(gu[:, :c.d_ff]) * gu[:, c.d_ff:]
            h = h + act @ np.asarray(w["w_down"], np.float64).T
        x = rmsnorm(h, np.asarray(self.glob["final_norm"], np.float64), c.rms_eps)
        return x @ np.asarray(self.glob["lm_head"], np.float64).T


def autoregressive_greedy(dec: Decoder, prompt: Sequence[int], n_new: int,
                          capacity: int = 0) -> List[int]:
    """Eq. 1 solved first to last: one token per forward, y_t = argmax P(y_t | y_<t, x)."""
    cache = dec.new_cache(capacity or len(prompt) + n_new + 1)
    out: List[int] = []
    nxt = None
    for t in prompt:
        logits = dec.forward_rows(cache, [int(t)], [-1])
        cache.seq_len += 1
        nxt = int(node_argmax(logits)[0])
    for _ in range(n_new):
        out.append(nxt)
        logits = dec.forward_rows(cache, [nxt], [-1])
        cache.seq_len += 1
        nxt = int(node_argmax(logits)[0])
    return out


def verify_step(dec: Decoder, cache: KVCache, tokens, parent):
    """One TR-Jacobi verification step (Section 3.3): forward, arg-max, acceptance, compaction.

    Returns a dict with the logits, the per-row prediction, k, path and bonus;
    the cache afterwards holds seq_len + k + 1 committed rows.
    """
    s = cache.seq_len
    logits = dec.forward_rows(cache, tokens, parent)
    pred = node_argmax(logits)
    k, path, bonus = accept_path(tokens, parent, pred)
    compact_rows(cache.k, s, path)
    cache.seq_len = compact_rows(cache.v, s, path)
    return {"logits": logits, "pred": pred, "k": k, "path": path, "bonus": bonus, "prefix": s}


def tr_jacobi_generate(dec: Decoder, prompt: Sequence[int], n_new: int, width: int,
                       n_branches: int, branch_len: int,
                       draw_fn: Callable[[int, int], Sequence[int]],
                       capacity: int = 0, trace: List[dict] = None) -> List[int]:
    """Greedy TR-Jacobi decoding (Section 3.3).

    The prompt is scored once (a chain tree over an empty cache), which yields
    the first committed token.  Every further step builds a tree from the
    current Jacobi window and the retrieved branches, verifies it in one
    forward and commits k + 1 tokens.  ``draw_fn(step, n)`` supplies the raw
    random integers behind ahead noise: step 0 seeds the first window; step
    t >= 1 uses slots [0, width) for the window refill after that step and
    slots [width, width + n_branches * branch_len) for that step's retrieval.
    When ``trace`` is a list, one record per step is appended to it.
    """
    n_tree = 1 + width + n_branches * branch_len
    cache = dec.new_cache(capacity or len(prompt) + n_new + n_tree + 1)
    p = len(prompt)
    logits = dec.forward_rows(cache, list(prompt), list(range(-1, p - 1)))
    cache.seq_len = p
    committed = [int(t) for t in prompt] + [int(node_argmax(logits[-1:])[0])]
    d0 = draw_fn(0, width)
    window = [ahead_noise(committed, d0[i]) for i in range(width)]
    step = 0
    while len(committed) - p < n_new:
        step += 1
        draws = draw_fn(step, width + n_branches * branch_len)
        branches = retrieve(committed, n_branches, branch_len, draws[width:])
        tokens, parent = build_tree(committed[-1], window, branches)
        rec = verify_step(dec, cache, tokens, parent)
        committed += [int(tokens[r]) for r in rec["path"][1:]] + [rec["bonus"]]
        window = refill_window(parent, rec["pred"], rec["path"][-1], width, committed, draws[:width])
        if trace is not None:
            rec.update(tokens=tokens, parent=parent, step=step, next_window=list(window))
            trace.append(rec)
    return committed[p:p + n_new]


def tr_jacobi_generate_tree(dec: Decoder, prompt: Sequence[int], n_new: int, parent: Sequence[int],
                            rank: Sequence[int], top_k: int, n_retrieved: int,
                            draw_fn: Callable[[int, int], Sequence[int]],
                            capacity: int = 0, trace: List[dict] = None) -> List[int]:
    """Greedy TR-Jacobi decoding over a static tree template with top-K siblings (Section 3.3, Appendix B).

    ``parent`` / ``rank`` describe the template (see ``refill_tree``); rows of rank -1 - j form one retrieval
    path of ``n_retrieved`` slots filled by prompt lookup.  All rows start as ahead noise (Section 3.3).
    ``draw_fn(step, n)``: step 0 seeds the first tree (slot i - 1 for row i); step t >= 1 uses slots [0, M - 1) for
    the refill after that step and slots [M - 1, M - 1 + n_retrieved) for that step's retrieval.
    """
    m = len(parent)
    cache = dec.new_cache(capacity or len(prompt) + n_new + m + 1)
    p = len(prompt)
    logits = dec.forward_rows(cache, list(prompt), list(range(-1, p - 1)))
    cache.seq_len = p
    committed = [int(t) for t in prompt] + [int(node_argmax(logits[-1:])[0])]
    d0 = draw_fn(0, m - 1)
    drafts = [ahead_noise(committed, d0[i]) for i in range(m - 1)]
    step = 0
    while len(committed) - p < n_new:
        step += 1
        draws = draw_fn(step, m - 1 + n_retrieved)
        retrieved = retrieve(committed, 1, n_retrieved, draws[m - 1:])[0] if n_retrieved else []
        tokens = np.asarray([committed[-1]] + list(drafts), np.int32)
        for i in range(1, m):                              # retrieval slots are refreshed from the current context
            if rank[i] < 0:
                tokens[i] = retrieved[-1 - rank[i]]
        rec = verify_step(dec, cache, tokens, parent)
        topk = node_topk(rec["logits"], top_k)
        committed += [int(tokens[r]) for r in rec["path"][1:]] + [rec["bonus"]]
        drafts = refill_tree(parent, rank, topk, rec["path"][-1], committed, draws[:m - 1],
                             retrieved if n_retrieved else [0])
        if trace is not None:
            rec.update(tokens=tokens, parent=np.asarray(parent, np.int32), step=step, topk=topk, next_drafts=list(drafts))
            trace.append(rec)
    return committed[p:p + n_new]
