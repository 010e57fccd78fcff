"""Helpers shared by the GPU parity tests: moving synthetic inputs to the device in libtrj's layouts."""
import numpy as np
import torch

import synth


def tdtype(dtype):
    return torch.bfloat16 if dtype == "bf16" else torch.float32


def to_dev(arr, dtype):
    return torch.from_numpy(np.ascontiguousarray(arr)).to("cuda", tdtype(dtype)).contiguous()


def i32(arr):
    return torch.from_numpy(np.ascontiguousarray(arr, dtype=np.int32)).cuda()


def anc_dev(anc):
    return torch.from_numpy(np.ascontiguousarray(anc).view(np.int64)).cuda()


class AttnCase:
    """A ragged batch of (prefix, tree) attention problems in device layout plus the host originals."""

    def __init__(self, trj, seed, n_heads, head_dim, prefixes, rows, parents, dtype="bf16", max_seq=None, pad=0,
                 kv_heads=0):
        self.h, self.d, self.dtype = n_heads, head_dim, dtype
        self.hk = kv_heads or n_heads
        self.prefixes, self.rows, self.parents = list(prefixes), list(rows), parents
        b = len(prefixes)
        self.max_len = max(s + m for s, m in zip(prefixes, rows))
        self.max_seq = max_seq or (self.max_len + pad)
        self.max_rows = max(rows)
        self.host = [synth.qkv(seed, n_heads, head_dim, s, m, dtype, name=f"seq{i}.", kv_heads=kv_heads)
                     for i, (s, m) in enumerate(zip(prefixes, rows))]
        # cache rows past the end of a sequence hold NaN: whatever a kernel fetches from there must not reach its output
        k = np.full((b, self.hk, self.max_seq, head_dim), np.nan, np.float32)
        v = np.full_like(k, np.nan)
        for i, (s, m) in enumerate(zip(prefixes, rows)):
            t = self.host[i]
            k[i, :, :s], v[i, :, :s] = t["k_prefix"], t["v_prefix"]
            k[i, :, s:s + m], v[i, :, s:s + m] = t["k_tree"], t["v_tree"]
        self.k, self.v = to_dev(k, dtype), to_dev(v, dtype)
        self.q = to_dev(np.concatenate([t["q"] for t in self.host], 0), dtype)
        words = 2
        anc = [trj.tree_from_parents(p, words)[1] for p in parents]
        self.depth = np.concatenate([trj.tree_from_parents(p, words)[0] for p in parents])
        self.anc = anc_dev(np.concatenate(anc, 0))
        self.seq_len = i32(prefixes)
        self.row_off_host = np.concatenate([[0], np.cumsum(rows)]).astype(np.int32)
        self.row_off = i32(self.row_off_host)

    def run(self, trj, **kw):
        return trj.tree_attention(self.q, self.k, self.v, self.seq_len, self.row_off, self.anc,
                                  max_rows=self.max_rows, max_len=self.max_len, **kw)

    def oracle_rows(self, oracle, seq, heads=None):
        """fp64 reference [M, len(heads), D] of sequence ``seq`` restricted to ``heads``."""
        t = self.host[seq]
        hs = list(range(self.h)) if heads is None else list(heads)
        ks = [h // (self.h // self.hk) for h in hs]          # the K/V head each of the chosen query heads reads
        return oracle.tree_attention(t["q"][:, hs], t["k_prefix"][ks], t["v_prefix"][ks],
                                     t["k_tree"][ks], t["v_tree"][ks], self.parents[seq])
