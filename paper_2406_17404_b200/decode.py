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

from . import Model, refill_window, retrieve


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
