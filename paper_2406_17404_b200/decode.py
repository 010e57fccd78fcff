"""Greedy TR-Jacobi decoding loop on top of the C ABI (host driver; integers only on the host).

Every step is one ``trj_step_host`` call (tree build, H2D, verification forward, acceptance, KV
compaction, D2H); retrieval and window refill are the library's host functions.  Random draws
behind ahead noise are supplied by the caller: ``draw_fn(step, n)`` returns n non-negative ints;
step 0 seeds the first window, step t >= 1 uses slots [0, width) for the refill after that step
and slots [width, width + n_branches * branch_len) for that step's retrieval.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import numpy as np

from . import Model, refill_tree, refill_window, retrieve, tree_from_parents


def upload_weights(cfg, layers, glob, device="cuda"):
    """numpy weight dicts (float32 values) -> CUDA tensors of the config's storage type."""
    import torch
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32

    def conv(name, arr):
        t = torch.from_numpy(np.ascontiguousarray(arr))
        return t.to(device=device, dtype=torch.float32 if "norm" in name else dt).contiguous()
    return ([{k: conv(k, v) for k, v in lw.items()} for lw in layers], {k: conv(k, v) for k, v in glob.items()})


def tr_jacobi_generate(model: Model, prompt: Sequence[int], n_new: int, width: int, n_branches: int,
                       branch_len: int, draw_fn: Callable[[int, int], Sequence[int]],
                       trace: Optional[List[dict]] = None) -> List[int]:
    """Decode ``n_new`` tokens after ``prompt`` for sequence 0 of ``model``; returns the new tokens."""
    import torch
    p = len(prompt)
    model.seq_len.zero_()
    toks = torch.tensor(np.asarray(prompt, np.int32), device=model.device)
    first = model.prefill(toks, 0)
    committed = [int(t) for t in prompt] + [int(first.item())]
    d0 = np.asarray(draw_fn(0, width), np.int64)
    window = np.array([committed[int(d) % len(committed)] for d in d0], np.int32)
    n_tree = 1 + width + n_branches * branch_len
    step = 0
    while len(committed) - p < n_new:
        step += 1
        draws = np.asarray(draw_fn(step, width + n_branches * branch_len), np.int64)
        branches = retrieve(committed, n_branches, branch_len, draws[width:])
        res = model.step_host(committed[-1], window, branches, max_len=len(committed) - 1 + n_tree)
        committed += [int(res["tokens"][r]) for r in res["path"][1:]] + [int(res["bonus"])]
        window = refill_window(res["parent"], res["node_argmax"], int(res["path"][-1]), width, committed, draws[:width])
        if trace is not None:
            res.update(step=step, next_window=window.copy())
            trace.append(res)
    return committed[p:p + n_new]


def tr_jacobi_generate_tree(model: Model, prompt: Sequence[int], n_new: int, parent: Sequence[int], rank: Sequence[int],
                            top_k: int, n_retrieved: int, draw_fn: Callable[[int, int], Sequence[int]],
                            trace: Optional[List[dict]] = None) -> List[int]:
    """Greedy TR-Jacobi decoding over a static tree template with top-K siblings (``parent`` / ``rank`` as for
    ``refill_tree``; rows of negative rank form one retrieval path of ``n_retrieved`` slots).  Per step: verification
    forward, per-row top-K, acceptance and KV compaction on the device; the integer refill on the host.
    ``draw_fn(step, n)``: step 0 seeds the first tree; step t >= 1 uses slots [0, M - 1) for the refill after that
    step and slots [M - 1, M - 1 + n_retrieved) for that step's retrieval."""
    import torch
    parent = np.ascontiguousarray(parent, np.int32)
    rank = np.ascontiguousarray(rank, np.int32)
    m, p, dev = len(parent), len(prompt), model.device
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    depth, anc = tree_from_parents(parent)
    d_par, d_dep, d_off = i32(parent), i32(depth), i32([0, m])
    d_anc = torch.from_numpy(anc.view(np.int64)).to(dev)
    model.seq_len.zero_()
    first = model.prefill(i32(prompt), 0)
    committed = [int(t) for t in prompt] + [int(first.item())]
    d0 = np.asarray(draw_fn(0, m - 1), np.int64)
    drafts = np.array([committed[int(d) % len(committed)] for d in d0], np.int32)
    step = 0
    while len(committed) - p < n_new:
        step += 1
        draws = np.asarray(draw_fn(step, m - 1 + n_retrieved), np.int64)
        retrieved = retrieve(committed, 1, n_retrieved, draws[m - 1:])[0] if n_retrieved else np.zeros(0, np.int32)
        tokens = np.concatenate([[committed[-1]], drafts]).astype(np.int32)
        slots = np.nonzero(rank < 0)[0]
        tokens[slots] = retrieved[-1 - rank[slots]]         # retrieval slots are refreshed from the current context
        d_tok = i32(tokens)
        out = model.verify_step(d_tok, d_par, d_dep, d_anc, d_off, max_rows=m, max_len=len(committed) - 1 + m)
        topk = model.node_topk(m, top_k)
        acc = model.accept(d_tok, d_par, d_dep, d_off, out["node_argmax"])
        model.compact_kv(acc["k_acc"], acc["path"])
        k = int(acc["k_acc"][0])
        path = acc["path"][0, :k + 1].cpu().numpy()
        committed += [int(tokens[r]) for r in path[1:]] + [int(acc["bonus"][0])]
        topk_h = topk.cpu().numpy()
        drafts = refill_tree(parent, rank, topk_h, int(path[-1]), committed, draws[:m - 1], retrieved)
        if trace is not None:
            trace.append({"step": step, "tokens": tokens, "k_acc": k, "path": path, "bonus": int(acc["bonus"][0]),
                          "topk": topk_h, "node_argmax": out["node_argmax"].cpu().numpy()})
    return committed[p:p + n_new]
