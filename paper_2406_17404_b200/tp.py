"""Tensor-parallel verification step: the decoder's heads and feed-forward columns split over ranks.

Every rank owns a ``Model`` built from its slice of the weights (``shard_weights``) and walks the step segment by
segment (trj_tp_begin / trj_tp_segment / trj_tp_finish); between two segments the ranks' partial sums of the half's
output projection are added by an all-reduce over the process group (NCCL across GPUs).  This module only cuts
tensors and orders calls: every arithmetic step of the decoder runs in the library's kernels, the sum over ranks
in the collective.
"""
from __future__ import annotations

from dataclasses import replace
from typing import Callable, Dict, List, Sequence, Tuple


def shard_cfg(cfg, world: int):
    """The shape of one rank's slice: heads, K/V heads and feed-forward width divided by ``world``."""
    kv = getattr(cfg, "n_kv_heads", 0) or cfg.n_heads
    if world < 1 or cfg.n_heads % world or kv % world or cfg.d_ff % world:
        raise ValueError(f"{world} ranks do not divide {cfg.n_heads} heads / {kv} K/V heads / d_ff {cfg.d_ff}")
    return replace(cfg, n_heads=cfg.n_heads // world, n_kv_heads=kv // world, d_ff=cfg.d_ff // world)


def shard_layer(cfg, layer: Dict[str, "object"], rank: int, world: int) -> Dict[str, "object"]:
    """Rank ``rank``'s slice of one layer's tensors (named as in trj_weights), as contiguous copies:
    wqkv rows of its query heads, then of its key heads, then of its value heads; wo columns of its heads;
    its gate rows then its up rows; its columns of w_down; the norm gains whole."""
    import torch
    D = cfg.head_dim
    kv = getattr(cfg, "n_kv_heads", 0) or cfg.n_heads
    hq, hk, f = cfg.n_heads // world, kv // world, cfg.d_ff // world
    HD, KD = cfg.n_heads * D, kv * D
    wqkv = layer["wqkv"]
    q = wqkv[rank * hq * D:(rank + 1) * hq * D]
    k = wqkv[HD + rank * hk * D:HD + (rank + 1) * hk * D]
    v = wqkv[HD + KD + rank * hk * D:HD + KD + (rank + 1) * hk * D]
    gu = layer["w_gate_up"]
    return {
        "attn_norm": layer["attn_norm"], "mlp_norm": layer["mlp_norm"],
        "wqkv": torch.cat([q, k, v], 0).contiguous(),
        "wo": layer["wo"][:, rank * hq * D:(rank + 1) * hq * D].contiguous(),
        "w_gate_up": torch.cat([gu[rank * f:(rank + 1) * f], gu[cfg.d_ff + rank * f:cfg.d_ff + (rank + 1) * f]], 0).contiguous(),
        "w_down": layer["w_down"][:, rank * f:(rank + 1) * f].contiguous(),
    }


def shard_weights(cfg, layers: Sequence[Dict[str, "object"]], glob: Dict[str, "object"], rank: int, world: int):
    """(cfg, layers, glob) of rank ``rank``; embedding, final norm and LM head are shared whole."""
    return shard_cfg(cfg, world), [shard_layer(cfg, l, rank, world) for l in layers], glob


def group_all_reduce(group=None) -> Callable[["object"], None]:
    """The sum over the ranks of a torch.distributed process group, in place."""
    import torch.distributed as dist

    def all_reduce(t) -> None:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return all_reduce


class TPRank:
    """One rank of a tensor-parallel decoder: its slice of the model plus the collective that adds the ranks'
    partial sums in place (``group_all_reduce()`` in a torch.distributed job)."""

    def __init__(self, model, all_reduce: Callable[["object"], None]):
        self.model, self.all_reduce = model, all_reduce

    def verify_step(self, tokens, parent, depth, anc, row_off, *, max_rows: int, max_len: int,
                    want_logits: bool = False, want_margin: bool = False, stream=None):
        """The verification step over the ranks: dict(node_argmax, margin | None, logits | None), equal on every rank."""
        m = self.model
        m.tp_begin(tokens, parent, depth, anc, row_off, max_rows=max_rows, max_len=max_len, stream=stream)
        n = m.tp_segments()
        for s in range(n):
            m.tp_segment(s, stream=stream)
            if s + 1 < n:
                self.all_reduce(m.tp_exchange_tensor())
        return m.tp_finish(want_logits=want_logits, want_margin=want_margin, stream=stream)


def _chain_chunks(model, tokens):
    """A prompt as chain trees of at most max_rows rows: (tokens, parent, depth, anc, row_off) device tensors."""
    import numpy as np
    import torch
    from . import tree_from_parents
    dev, n = model.device, tokens.numel()
    for lo in range(0, n, model.max_rows):
        m = min(model.max_rows, n - lo)
        parent = np.arange(-1, m - 1, dtype=np.int32)
        depth, anc = tree_from_parents(parent)
        as_dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dev, dt)
        yield (tokens[lo:lo + m].to(dev, torch.int32).contiguous(), as_dev(parent, torch.int32), as_dev(depth, torch.int32),
               as_dev(anc.view(np.int64), torch.int64), torch.tensor([0, m], dtype=torch.int32, device=dev))


def prefill(rank: "TPRank", tokens):
    """Scores a prompt (sequence 0) chunk by chunk as chain trees; every row stays where the step wrote it.
    Returns the device tensor holding the first greedy token."""
    m, out = rank.model, None
    for tok, parent, depth, anc, off in _chain_chunks(m, tokens):
        rows = tok.numel()
        out = rank.verify_step(tok, parent, depth, anc, off, max_rows=rows, max_len=m.max_seq)
        m.seq_len[:1] += rows
    return out["node_argmax"][-1:]


def prefill_local(models: List["object"], tokens):
    """``prefill`` for ranks that share one device (see verify_step_local)."""
    out = None
    for tok, parent, depth, anc, off in _chain_chunks(models[0], tokens):
        rows = tok.numel()
        out = verify_step_local(models, tok, parent, depth, anc, off, max_rows=rows, max_len=models[0].max_seq)
        for m in models:
            m.seq_len[:1] += rows
    return out[0]["node_argmax"][-1:]


def verify_step_local(models: List["object"], tokens, parent, depth, anc, row_off, *, max_rows: int, max_len: int,
                      want_logits: bool = False, want_margin: bool = False) -> List[Dict[str, "object"]]:
    """All ranks' contexts on ONE device, stepped in lock-step on the current stream; the collective is a plain sum
    of the exchange buffers in rank order, written back to every rank.  For checking a sharding on a single
    device: nothing here runs concurrently, so no kernel waits on another rank."""
    for m in models:
        m.tp_begin(tokens, parent, depth, anc, row_off, max_rows=max_rows, max_len=max_len)
    n = models[0].tp_segments()
    for s in range(n):
        for m in models:
            m.tp_segment(s)
        if s + 1 < n:
            bufs = [m.tp_exchange_tensor() for m in models]
            total = bufs[0].clone()
            for b in bufs[1:]:
                total += b
            for b in bufs:
                b.copy_(total)
    return [m.tp_finish(want_logits=want_logits, want_margin=want_margin) for m in models]
