"""Seeded synthetic inputs for the TR-Jacobi verification step.

This module only *draws data*: model weights, prompts, tree topologies, q/k/v
tensors, logits and draft tokens.  It holds none of the method's arithmetic
(no attention, no mask construction, no acceptance rule, no compaction), so
both the CPU oracle and the CUDA path can be fed from it without sharing any
code of the method itself.

Every draw is keyed by ``(seed, name)`` through a counter-based Philox stream,
so two callers asking for the same tensor get identical values regardless of
the order in which they ask.

Floating-point tensors are returned as ``float32`` arrays.  When a config is
bf16 the values are first rounded to the nearest bf16 (ties to even), so the
same array widened to fp64 on the CPU and narrowed to bf16 on the GPU
represents exactly the same numbers.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

__all__ = [
    "ModelCfg", "TINY", "TINY_GQA", "LLAMA7B", "LLAMA3_8B", "stream", "round_bf16", "bf16_bits",
    "layer_weights", "global_weights", "prompt", "chain_parents",
    "random_tree", "tree_template", "node_depths", "qkv", "logits", "planted_tokens",
    "random_path", "ragged_batch", "noise_draws",
]


# --------------------------------------------------------------------------
# configs
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class ModelCfg:
    """LLaMA-family decoder shape (RMSNorm, RoPE, MHA or grouped-query attention, SwiGLU, untied LM head).

    ``n_kv_heads`` = 0 means one K/V head per query head; otherwise query head h uses K/V head
    h // (n_heads // n_kv_heads)."""
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    dtype: str = "bf16"          # "bf16" | "f32": storage type of weights/activations
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    weight_std: float = 0.02
    n_kv_heads: int = 0

    @property
    def kv_heads(self) -> int:
        return self.n_kv_heads or self.n_heads

    def with_layers(self, n: int) -> "ModelCfg":
        return replace(self, n_layers=n)


TINY = ModelCfg(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ff=688,
                vocab=1024, dtype="f32")
TINY_GQA = ModelCfg(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ff=688,
                    vocab=1024, dtype="f32", n_kv_heads=2)
LLAMA7B = ModelCfg(n_layers=32, d_model=4096, n_heads=32, head_dim=128,
                   d_ff=11008, vocab=32000, dtype="bf16")
# the shape of the paper's main model family (Table 2): grouped-query attention with 8 K/V heads, 128 256-way vocabulary
LLAMA3_8B = ModelCfg(n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ff=14336, vocab=128256,
                     dtype="bf16", rope_theta=500000.0, n_kv_heads=8)


# --------------------------------------------------------------------------
# random streams and bf16 rounding
# --------------------------------------------------------------------------
def stream(seed: int, name: str) -> np.random.Generator:
    """Independent Philox stream for ``(seed, name)``."""
    h = hashlib.blake2b(f"{seed}:{name}".encode(), digest_size=16).digest()
    key = np.frombuffer(h, dtype=np.uint64).copy()
    return np.random.Generator(np.random.Philox(key=key))


def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    r = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    r &= np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Upper 16 bits of float32 values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def _normal(seed: int, name: str, shape, std: float, dtype: str) -> np.ndarray:
    g = stream(seed, name)
    x = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return round_bf16(x) if dtype == "bf16" else x


# --------------------------------------------------------------------------
# model weights (random init; norm gains are 1)
# --------------------------------------------------------------------------
def layer_weights(cfg: ModelCfg, seed: int, layer: int) -> Dict[str, np.ndarray]:
    """Weights of one decoder layer.  Every matrix is [d_out, d_in] (d_in contiguous).

    ``wqkv`` stacks the query, key and value projections (rows 0..q-1 = Wq,
    q..q+kv-1 = Wk, q+kv..q+2kv-1 = Wv, q = n_heads*head_dim, kv = kv_heads*head_dim);
    ``w_gate_up`` stacks the SwiGLU gate rows (0..f-1) over the up rows (f..2f-1).
    """
    d, f, hd = cfg.d_model, cfg.d_ff, cfg.n_heads * cfg.head_dim
    kvd = cfg.kv_heads * cfg.head_dim
    s, t = cfg.weight_std, cfg.dtype
    p = f"layer{layer}."
    return {
        "attn_norm": np.ones(d, np.float32),
        "wqkv": _normal(seed, p + "wqkv", (hd + 2 * kvd, d), s, t),
        "wo": _normal(seed, p + "wo", (d, hd), s, t),
        "mlp_norm": np.ones(d, np.float32),
        "w_gate_up": _normal(seed, p + "w_gate_up", (2 * f, d), s, t),
        "w_down": _normal(seed, p + "w_down", (d, f), s, t),
    }


def global_weights(cfg: ModelCfg, seed: int) -> Dict[str, np.ndarray]:
    """Embedding table [V, d], untied LM head [V, d] and the final norm gain."""
    return {
        "embed": _normal(seed, "embed", (cfg.vocab, cfg.d_model), cfg.weight_std, cfg.dtype),
        "lm_head": _normal(seed, "lm_head", (cfg.vocab, cfg.d_model), cfg.weight_std, cfg.dtype),
        "final_norm": np.ones(cfg.d_model, np.float32),
    }


def prompt(seed: int, n: int, vocab: int) -> np.ndarray:
    """``n`` token ids drawn uniformly from [0, vocab)."""
    return stream(seed, "prompt").integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)


# --------------------------------------------------------------------------
# tree topologies (parent pointers only; masks are built by each side itself)
# --------------------------------------------------------------------------
def chain_parents(m: int) -> np.ndarray:
    """Row 0 is the root (parent -1); row i hangs off row i-1."""
    return np.arange(-1, m - 1, dtype=np.int32)


def node_depths(parent: np.ndarray) -> np.ndarray:
    """Number of edges from the root, following parent pointers (parent[i] < i)."""
    depth = np.zeros(len(parent), np.int32)
    for i in range(1, len(parent)):
        depth[i] = depth[parent[i]] + 1
    return depth


def random_tree(seed: int, m: int, max_depth: int, max_children: int,
                name: str = "tree") -> np.ndarray:
    """Random topologically-ordered tree with ``m`` rows (row 0 = root).

    Row i >= 1 draws its parent uniformly among the earlier rows whose depth is
    below ``max_depth`` and which still have fewer than ``max_children``
    children.  The first ``max_depth`` rows after the root form a chain so the
    stated depth is always reached.
    """
    g = stream(seed, name)
    parent = np.full(m, -1, np.int32)
    depth = np.zeros(m, np.int32)
    nchild = np.zeros(m, np.int32)
    for i in range(1, m):
        if i <= max_depth:
            p = i - 1
        else:
            ok = np.nonzero((depth[:i] < max_depth) & (nchild[:i] < max_children))[0]
            if len(ok) == 0:
                raise ValueError("tree parameters admit no further node")
            p = int(ok[g.integers(0, len(ok))])
        parent[i] = p
        depth[i] = depth[p] + 1
        nchild[p] += 1
    return parent


def tree_template(seed: int, n_nodes: int = 63, max_depth: int = 4, first_level: int = 10,
                  retrieval_len: int = 5, name: str = "template") -> Tuple[np.ndarray, np.ndarray]:
    """A seeded sparse tree template with top-K siblings plus one retrieval path (stands in for the paper's
    third-party 63-node template, which is not printed there): returns (parent[M], rank[M]), M = 1 + n_nodes +
    retrieval_len, row 0 the root.

    Rows are added one at a time as the next-ranked child of a drawn parent (the root has up to ``first_level``
    children, every other row up to 3; depth <= ``max_depth``), parents being drawn with a weight that halves with
    every level and shrinks with every child already present (x 0.8 at the root, x 0.5 elsewhere), so the tree is
    wide near the root and sparse below it.  The
    rank of a row is its position among its siblings (0 = most likely candidate).  The retrieval path is a chain
    off the root whose rows carry rank -1 - j (slot j).  Rows are then renumbered level by level so that
    parent[i] < i and rank-0 children come first.
    """
    g = stream(seed, name)
    parent, depth, nchild = [-1], [0], [0]
    rank = [0]
    for _ in range(n_nodes):
        cap = [first_level if i == 0 else 3 for i in range(len(parent))]
        w = np.array([0.0 if (depth[i] >= max_depth or nchild[i] >= cap[i])
                      else 0.5 ** depth[i] * (0.8 if i == 0 else 0.5) ** nchild[i] for i in range(len(parent))])
        p = int(g.choice(len(parent), p=w / w.sum()))
        parent.append(p); depth.append(depth[p] + 1); rank.append(nchild[p]); nchild.append(0)
        nchild[p] += 1
    prev = 0
    for j in range(retrieval_len):
        parent.append(prev); depth.append(depth[prev] + 1); rank.append(-1 - j); nchild.append(0)
        prev = len(parent) - 1
    # renumber: breadth-first, siblings by rank (retrieval rows last among the root's children)
    order = sorted(range(len(parent)), key=lambda i: (depth[i], parent[i] if parent[i] >= 0 else -1,
                                                      rank[i] if rank[i] >= 0 else 1000 - rank[i]))
    # a stable breadth-first order needs parents renumbered first: do it level by level
    new_of = {0: 0}
    out_parent, out_rank = [-1], [0]
    for d in range(1, max(depth) + 1):
        level = [i for i in order if depth[i] == d]
        level.sort(key=lambda i: (new_of[parent[i]], rank[i] if rank[i] >= 0 else 1000 - rank[i]))
        for i in level:
            new_of[i] = len(out_parent)
            out_parent.append(new_of[parent[i]])
            out_rank.append(rank[i])
    return np.asarray(out_parent, np.int32), np.asarray(out_rank, np.int32)


# --------------------------------------------------------------------------
# op-level tensors
# --------------------------------------------------------------------------
def qkv(seed: int, n_heads: int, head_dim: int, prefix: int, rows: int,
        dtype: str = "bf16", name: str = "", kv_heads: int = 0) -> Dict[str, np.ndarray]:
    """q/k/v ~ N(0,1).  q: [rows, H, D]; k/v prefix: [Hkv, prefix, D]; k/v tree: [Hkv, rows, D] (Hkv = H unless
    ``kv_heads`` says otherwise)."""
    n = name
    hk = kv_heads or n_heads
    return {
        "q": _normal(seed, n + "q", (rows, n_heads, head_dim), 1.0, dtype),
        "k_prefix": _normal(seed, n + "k_prefix", (hk, prefix, head_dim), 1.0, dtype),
        "v_prefix": _normal(seed, n + "v_prefix", (hk, prefix, head_dim), 1.0, dtype),
        "k_tree": _normal(seed, n + "k_tree", (hk, rows, head_dim), 1.0, dtype),
        "v_tree": _normal(seed, n + "v_tree", (hk, rows, head_dim), 1.0, dtype),
    }


def logits(seed: int, rows: int, vocab: int, dtype: str = "bf16", name: str = "logits") -> np.ndarray:
    """[rows, vocab] ~ N(0,1)."""
    return _normal(seed, name, (rows, vocab), 1.0, dtype)


def planted_tokens(seed: int, parent: np.ndarray, row_best: np.ndarray, vocab: int,
                   p_hit: float = 0.6, name: str = "plant") -> np.ndarray:
    """Draft token of every row, with a controlled hit rate.

    ``row_best[i]`` is the id the caller found to have the largest logit in row
    i.  With probability ``p_hit`` row j carries exactly the id its parent
    predicts (``row_best[parent[j]]``), otherwise a different uniformly drawn
    id, so accepted path lengths spread over 0..depth instead of always 0.
    The root's token is a uniform draw.
    """
    g = stream(seed, name)
    m = len(parent)
    tok = g.integers(0, vocab, size=m, dtype=np.int64).astype(np.int32)
    hit = g.random(m) < p_hit
    for j in range(1, m):
        want = int(row_best[parent[j]])
        if hit[j]:
            tok[j] = want
        elif tok[j] == want:
            tok[j] = (want + 1) % vocab
    return tok


def random_path(seed: int, parent: np.ndarray, k: int, name: str = "path") -> np.ndarray:
    """Rows of a root-to-node path ending at a uniformly drawn node of depth ``k``."""
    depth = node_depths(parent)
    cand = np.nonzero(depth == k)[0]
    if len(cand) == 0:
        raise ValueError(f"no node of depth {k}")
    node = int(cand[stream(seed, name).integers(0, len(cand))])
    rows: List[int] = []
    while node >= 0:
        rows.append(node)
        node = int(parent[node])
    return np.asarray(rows[::-1], np.int32)


def ragged_batch(seed: int, batch: int, prefix_range: Tuple[int, int],
                 rows_range: Tuple[int, int]) -> Tuple[np.ndarray, np.ndarray]:
    """Per-sequence prefix lengths and tree sizes, uniform on the closed ranges."""
    g = stream(seed, "ragged")
    s = g.integers(prefix_range[0], prefix_range[1] + 1, size=batch).astype(np.int32)
    m = g.integers(rows_range[0], rows_range[1] + 1, size=batch).astype(np.int32)
    return s, m


def noise_draws(seed: int, step: int, n: int) -> np.ndarray:
    """``n`` raw non-negative random integers for decode step ``step`` (ahead-noise sampling)."""
    return stream(seed, f"noise{step}").integers(0, 2 ** 31 - 1, size=n, dtype=np.int64)
