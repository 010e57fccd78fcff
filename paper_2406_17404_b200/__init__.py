"""Python binding of libtrj: the TR-Jacobi verification step on one B200.

Argument marshalling only: every function here checks tensor types, passes
device pointers to the C ABI declared in ``include/trj.h`` and returns torch
tensors (PyTorch supplies device memory and streams, nothing else).  There is
no fallback: if ``libtrj.so`` is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtrj.so")

MAX_ROWS = 128
MAX_BATCH = 64
MAX_TOPK = 10
PATH_STRIDE = 128
# bytes trj_step_host moves per call: tokens/parent/depth/row_off + ancestor words in, predictions/k/bonus/path out
STEP_H2D_BYTES = (3 * MAX_ROWS + 4) * 4 + MAX_ROWS * 2 * 8
STEP_D2H_BYTES = (MAX_ROWS + 2 + PATH_STRIDE + 2) * 4      # ... and the two device status words
F32, BF16 = 0, 1

_lib = None


class TrjError(RuntimeError):
    """A libtrj call returned a non-zero status."""

    def __init__(self, status: int, message: str):
        super().__init__(f"libtrj status {status}: {message}")
        self.status = status


class ModelCfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ff", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int32) for n in ("dtype", "max_batch", "max_seq", "max_rows", "n_kv_heads")]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("attn_norm", C.POINTER(C.c_void_p)), ("wqkv", C.POINTER(C.c_void_p)),
                ("wo", C.POINTER(C.c_void_p)), ("mlp_norm", C.POINTER(C.c_void_p)),
                ("w_gate_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p))]


_I32P, _I64P, _U64P = C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.POINTER(C.c_uint64)
_VP, _I, _SZ = C.c_void_p, C.c_int32, C.c_size_t

# name -> (restype, argtypes); mirrors include/trj.h one to one
_SIGNATURES = {
    "trj_last_error": (C.c_char_p, []),
    "trj_version": (C.c_char_p, []),
    "trj_build_tree": (_I, [_I, _I32P, _I, _I32P, _I, _I, _I, _I, _I32P, _I32P, _I32P, _U64P, _I32P]),
    "trj_tree_from_parents": (_I, [_I32P, _I, _I, _I32P, _U64P]),
    "trj_retrieve": (_I, [_I32P, _I, _I, _I, _I64P, _I32P]),
    "trj_refill_window": (_I, [_I32P, _I32P, _I, _I, _I, _I32P, _I, _I64P, _I32P]),
    "trj_tree_attention_workspace": (_SZ, [_I, _I, _I, _I, _I]),
    "trj_tree_attention": (_I, [_VP, _VP, _VP, _VP, _VP, _VP, _I, _I, _I, _I, _I, _I, _I, _I, _I, _VP, _VP, _SZ, _VP]),
    "trj_tree_attention_gqa": (_I, [_VP, _VP, _VP, _VP, _VP, _VP, _I, _I, _I, _I, _I, _I, _I, _I, _I, _I, _VP, _VP, _SZ, _VP]),
    "trj_argmax_accept_workspace": (_SZ, [_I, _I]),
    "trj_argmax_accept": (_I, [_VP, _I, _I, _VP, _VP, _VP, _VP, _I, _I, _VP, _VP, _VP, _VP, _VP, _VP, _SZ, _VP]),
    "trj_topk_accept_workspace": (_SZ, []),
    "trj_topk_accept": (_I, [_VP, _I, _I, _I, _VP, _VP, _VP, _VP, _I, _I, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _SZ, _VP]),
    "trj_node_topk": (_I, [_VP, _I, _I, _VP, _VP]),
    "trj_refill_tree": (_I, [_I32P, _I32P, _I, _I32P, _I, _I, _I32P, _I, _I64P, _I32P, _I, _I32P]),
    "trj_argmax_accept_static": (_I, [_VP, _I, _I, _VP, _VP, _VP, _VP, _I, _I, _VP, _VP, _VP, _VP, _VP, _VP]),
    "trj_compact_rows": (_I, [_VP, _VP, _I, _I, _I, _I, _I, _I, _VP, _VP, _VP, _VP]),
    "trj_workspace_bytes": (_SZ, [C.POINTER(ModelCfg)]),
    "trj_create": (_I, [C.POINTER(ModelCfg), C.POINTER(Weights), _VP, _SZ, C.POINTER(_VP)]),
    "trj_destroy": (_I, [_VP]),
    "trj_verify_step": (_I, [_VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _I, _VP, _I, _I, _I, _I, _VP, _VP, _VP, _VP]),
    "trj_tp_segments": (_I, [_VP]),
    "trj_tp_begin": (_I, [_VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _I, _VP, _I, _I, _I, _I, _VP]),
    "trj_tp_segment": (_I, [_VP, _I, _VP]),
    "trj_tp_exchange_buffer": (_I, [_VP, C.POINTER(_VP), C.POINTER(_SZ)]),
    "trj_tp_finish": (_I, [_VP, _VP, _VP, _VP, _VP]),
    "trj_accept": (_I, [_VP, _VP, _VP, _VP, _VP, _I, _I, _VP, _VP, _VP, _VP, _VP]),
    "trj_compact_kv": (_I, [_VP, _VP, _VP, _VP, _I, _VP, _VP, _VP]),
    "trj_prefill": (_I, [_VP, _VP, _VP, _VP, _I, _VP, _I, _VP, _VP]),
    "trj_step_host": (_I, [_VP, _VP, _VP, _VP, _I, _I, _I32P, _I, _I32P, _I, _I, _I32P, _I32P, _I32P, _I32P,
                           _I32P, _I32P, _I32P, _VP]),
    "trj_draft_tokens": (_I, [_VP, _VP, _VP, _I, _I, _I, _VP, _VP, _VP]),
    "trj_commit_refill": (_I, [_VP, _VP, _VP, _I, _VP, _VP, _VP, _VP, _I, _VP, _I, _VP, _VP, _VP, _VP]),
    "trj_decode_device": (_I, [_VP, _VP, _VP, _VP, _VP, _I, _VP, _I, _VP, _I, _I, _I, _VP, _I, _VP, _VP]),
    "trj_decode_device_tree": (_I, [_VP, _VP, _VP, _VP, _VP, _I, _VP, _I, _I32P, _I32P, _I, _I, _I, _VP, _VP, _I, _VP, _VP]),
    "trj_set_draft_source": (_I, [_VP, _VP, _I, _VP, _I]),
    "trj_gemm_workspace": (_SZ, [_I, _I, _I]),
    "trj_gemm": (_I, [_VP, _VP, _VP, _I, _I, _I, _I, _VP, _SZ, _VP]),
    "trj_device_status": (_I, [_VP, _I, _VP]),
    "trj_selftest_wait_expiry": (_I, [_VP, _I, _VP]),
    "trj_debug_flags": (_I, [_I32P]),
    "trj_timeline_reset": (_I, [_VP]),
    "trj_timeline_read": (_I, [_I, _I, _U64P, _U64P, _I32P]),
    "trj_timeline_ctas_per_sm": (_I, [_I32P]),
    "trj_launch_count": (C.c_uint64, []),
    "trj_set_pdl": (None, [_I]),
    "trj_profile_enable": (_I, [_VP, _I]),
    "trj_profile_read": (_I, [_VP, C.POINTER(C.c_float), _I32P, _I]),
}
PROF_CATEGORIES = ("elementwise", "gemm", "rope_kv", "attention", "argmax_accept", "compact")
EXPORTS = tuple(_SIGNATURES)


def use_library(path: str) -> None:
    """Load another build of the library (the clock-stamp build) instead of the default one; call before lib()."""
    global _lib, LIB_PATH
    if _lib is not None:
        raise RuntimeError("a library is already loaded")
    LIB_PATH = path


def debug_flags() -> int:
    """trj_debug_flags (debug build only): index-check bits seen since the last call."""
    f = C.c_int32(0)
    _check(lib().trj_debug_flags(C.byref(f)))
    return int(f.value)


TL_KINDS = ("rmsnorm", "gemm", "rope_kv", "attention", "swiglu", "embed")


def timeline_reset(stream=None) -> None:
    """trj_timeline_reset (clock-stamp build only)."""
    _check(lib().trj_timeline_reset(_stream(stream)))


def timeline_read(max_launches: int = 512):
    """trj_timeline_read for every kind: {kind: (begin_ns, end_ns)} as uint64 arrays in launch order."""
    out = {}
    for kind, name in enumerate(TL_KINDS):
        b, e = np.zeros(max_launches, np.uint64), np.zeros(max_launches, np.uint64)
        n = C.c_int32(0)
        _check(lib().trj_timeline_read(kind, max_launches, b.ctypes.data_as(_U64P), e.ctypes.data_as(_U64P), C.byref(n)))
        out[name] = (b[:n.value].copy(), e[:n.value].copy())
    return out


def timeline_ctas_per_sm() -> int:
    """trj_timeline_ctas_per_sm (clock-stamp build only)."""
    v = C.c_int32(0)
    _check(lib().trj_timeline_ctas_per_sm(C.byref(v)))
    return int(v.value)


def lib() -> C.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2406_17404_b200.build`; "
                              "there is no fallback path")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _check(status: int) -> None:
    if status != 0:
        raise TrjError(status, lib().trj_last_error().decode())


def version() -> str:
    return lib().trj_version().decode()


def set_pdl(on: bool) -> None:
    """trj_set_pdl: programmatic dependent launch of the step's kernels on (default) or off."""
    lib().trj_set_pdl(1 if on else 0)


def launch_count() -> int:
    """trj_launch_count: kernel launches enqueued by the library in this process."""
    return int(lib().trj_launch_count())


# ----------------------------------------------------------------------------- host helpers (numpy)
def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _p32(a: np.ndarray):
    return a.ctypes.data_as(_I32P)


def build_tree(root: int, window: Sequence[int], branches, max_rows: int = MAX_ROWS,
               anc_words: int = 2) -> Dict[str, np.ndarray]:
    """trj_build_tree: tokens, parent, depth [M] and anc [M, anc_words] of the merged tree."""
    window = _i32(window).reshape(-1)
    br = _i32(branches) if len(branches) else np.zeros((0, 0), np.int32)
    br = br.reshape(br.shape[0], -1) if br.ndim >= 1 and br.size else np.zeros((0, 0), np.int32)
    r, bl = (br.shape[0], br.shape[1]) if br.size else (0, 0)
    cap = max(1, min(max_rows, MAX_ROWS))
    tokens, parent, depth = (np.zeros(cap, np.int32) for _ in range(3))
    anc = np.zeros((cap, anc_words), np.uint64)
    n = C.c_int32(0)
    _check(lib().trj_build_tree(int(root), _p32(window), len(window), _p32(br), r, bl, max_rows, anc_words,
                                _p32(tokens), _p32(parent), _p32(depth), anc.ctypes.data_as(_U64P), C.byref(n)))
    m = n.value
    return {"tokens": tokens[:m], "parent": parent[:m], "depth": depth[:m], "anc": anc[:m]}


def tree_from_parents(parent, anc_words: int = 2) -> Tuple[np.ndarray, np.ndarray]:
    """trj_tree_from_parents: (depth [M], anc [M, anc_words])."""
    parent = _i32(parent)
    m = len(parent)
    depth = np.zeros(max(m, 1), np.int32)
    anc = np.zeros((max(m, 1), anc_words), np.uint64)
    _check(lib().trj_tree_from_parents(_p32(parent), m, anc_words, _p32(depth), anc.ctypes.data_as(_U64P)))
    return depth[:m], anc[:m]


def retrieve(context, n_branches: int, branch_len: int, draws) -> np.ndarray:
    """trj_retrieve: [n_branches, branch_len] retrieved (or noise) tokens."""
    context = _i32(context)
    draws = np.ascontiguousarray(draws, dtype=np.int64)
    out = np.zeros((n_branches, branch_len), np.int32)
    _check(lib().trj_retrieve(_p32(context), len(context), n_branches, branch_len,
                              draws.ctypes.data_as(_I64P), _p32(out)))
    return out


def refill_window(parent, node_argmax, best: int, width: int, context, draws) -> np.ndarray:
    """trj_refill_window: the next Jacobi window [width]."""
    parent, node_argmax, context = _i32(parent), _i32(node_argmax), _i32(context)
    draws = np.ascontiguousarray(draws, dtype=np.int64)
    out = np.zeros(max(width, 1), np.int32)
    _check(lib().trj_refill_window(_p32(parent), _p32(node_argmax), len(parent), int(best), width,
                                   _p32(context), len(context), draws.ctypes.data_as(_I64P), _p32(out)))
    return out[:width]


# ----------------------------------------------------------------------------- device entry points (torch)
def _torch():
    import torch
    return torch


def _dtype_code(t) -> int:
    torch = _torch()
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}: libtrj takes bfloat16 or float32")


def _dev(t, dtype=None, name="tensor"):
    torch = _torch()
    if not isinstance(t, torch.Tensor) or not t.is_cuda or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream(stream=None):
    torch = _torch()
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _scratch(nbytes: int, device, zero: bool = False):
    torch = _torch()
    n = max(256, int(nbytes))
    return (torch.zeros if zero else torch.empty)(n, dtype=torch.uint8, device=device)


def tree_attention_workspace(rows_total: int, batch: int, n_heads: int, head_dim: int, max_len: int) -> int:
    return int(lib().trj_tree_attention_workspace(rows_total, batch, n_heads, head_dim, max_len))


def tree_attention(q, k_cache, v_cache, seq_len, row_off, anc, *, max_rows: int, max_len: int,
                   out=None, workspace=None, stream=None):
    """trj_tree_attention (trj_tree_attention_gqa when the cache has fewer heads than q).  q [rows, H, D];
    k/v_cache [B, Hkv, max_seq, D]; seq_len [B]; row_off [B+1]; anc [rows, anc_words] (int64 view of the u64
    words).  Returns out [rows, H, D]."""
    torch = _torch()
    rows, n_heads, hd = q.shape
    batch, kv_heads, max_seq, _ = k_cache.shape
    if out is None:
        out = torch.empty_like(q)
    need = tree_attention_workspace(rows, batch, n_heads, hd, max_len)
    if workspace is None:
        workspace = _scratch(need, q.device)
    args = (_dev(q, name="q"), _dev(k_cache, q.dtype, "k_cache"), _dev(v_cache, q.dtype, "v_cache"),
            _dev(seq_len, torch.int32, "seq_len"), _dev(row_off, torch.int32, "row_off"), _dev(anc, torch.int64, "anc"),
            anc.shape[1], batch, rows, max_rows, n_heads)
    tail = (hd, max_seq, max_len, _dtype_code(q), _dev(out, q.dtype, "out"), _dev(workspace, torch.uint8, "workspace"),
            workspace.numel(), _stream(stream))
    if kv_heads == n_heads:
        _check(lib().trj_tree_attention(*args, *tail))
    else:
        _check(lib().trj_tree_attention_gqa(*args, kv_heads, *tail))
    return out


def argmax_accept_workspace(rows_total: int, batch: int) -> int:
    return int(lib().trj_argmax_accept_workspace(rows_total, batch))


def argmax_accept(logits, tokens, parent, depth, row_off, *, want_margin: bool = True, workspace=None, stream=None):
    """trj_argmax_accept.  logits [rows, V]; tokens/parent/depth [rows] int32; row_off [B+1] int32.
    Returns dict(node_argmax [rows], margin [rows] | None, k_acc [B], path [B, PATH_STRIDE], bonus [B]).
    ``workspace`` must be zero-filled before its first use (a fresh one is zeroed here)."""
    torch = _torch()
    rows, vocab = logits.shape
    batch = row_off.numel() - 1
    dev = logits.device
    if workspace is None:
        workspace = _scratch(argmax_accept_workspace(rows, batch), dev, zero=True)
    i32 = dict(dtype=torch.int32, device=dev)
    node_argmax = torch.empty(rows, **i32)
    margin = torch.empty(rows, dtype=torch.float32, device=dev) if want_margin else None
    k_acc, bonus = torch.empty(batch, **i32), torch.empty(batch, **i32)
    path = torch.empty(batch, PATH_STRIDE, **i32)
    _check(lib().trj_argmax_accept(
        _dev(logits, name="logits"), _dtype_code(logits), vocab, _dev(tokens, torch.int32, "tokens"),
        _dev(parent, torch.int32, "parent"), _dev(depth, torch.int32, "depth"), _dev(row_off, torch.int32, "row_off"),
        batch, rows, _dev(node_argmax), _dev(margin) if want_margin else None, _dev(k_acc), _dev(path), _dev(bonus),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)))
    return {"node_argmax": node_argmax, "margin": margin, "k_acc": k_acc, "path": path, "bonus": bonus}


def topk_accept(logits, tokens, parent, depth, row_off, k: int, *, workspace=None, stream=None):
    """trj_topk_accept: :func:`argmax_accept` plus ``topk`` [rows, k] int32, the ids of every row's k largest logits."""
    torch = _torch()
    rows, vocab = logits.shape
    batch = row_off.numel() - 1
    dev = logits.device
    if workspace is None:
        workspace = _scratch(lib().trj_topk_accept_workspace(), dev, zero=True)
    i32 = dict(dtype=torch.int32, device=dev)
    topk, node_argmax = torch.empty(rows, k, **i32), torch.empty(rows, **i32)
    margin = torch.empty(rows, dtype=torch.float32, device=dev)
    k_acc, bonus, path = torch.empty(batch, **i32), torch.empty(batch, **i32), torch.empty(batch, PATH_STRIDE, **i32)
    _check(lib().trj_topk_accept(
        _dev(logits, name="logits"), _dtype_code(logits), vocab, int(k), _dev(tokens, torch.int32, "tokens"),
        _dev(parent, torch.int32, "parent"), _dev(depth, torch.int32, "depth"), _dev(row_off, torch.int32, "row_off"),
        batch, rows, _dev(topk), _dev(node_argmax), _dev(margin), _dev(k_acc), _dev(path), _dev(bonus),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)))
    return {"topk": topk, "node_argmax": node_argmax, "margin": margin, "k_acc": k_acc, "path": path, "bonus": bonus}


def refill_tree(parent, rank, topk, best: int, context, draws, retrieved=()) -> np.ndarray:
    """trj_refill_tree: draft tokens [M - 1] of the next step for a template with top-K siblings (host)."""
    parent, rank, context = _i32(parent), _i32(rank), _i32(context)
    topk = _i32(topk).reshape(len(parent), -1)
    draws = np.ascontiguousarray(draws, dtype=np.int64)
    retrieved = _i32(retrieved).reshape(-1)
    out = np.zeros(max(len(parent) - 1, 1), np.int32)
    _check(lib().trj_refill_tree(_p32(parent), _p32(rank), len(parent), _p32(topk), topk.shape[1], int(best),
                                 _p32(context), len(context), draws.ctypes.data_as(_I64P),
                                 _p32(retrieved) if len(retrieved) else None, len(retrieved), _p32(out)))
    return out[:len(parent) - 1]


def argmax_accept_into(logits, tokens, parent, depth, row_off, out, workspace, *, stream=None) -> None:
    """trj_argmax_accept into preallocated outputs (``out`` as for :func:`argmax_accept_static`) with a caller-held,
    zero-initialised workspace: nothing is allocated, so the call can be captured in a CUDA graph."""
    torch = _torch()
    rows, vocab = logits.shape
    batch = row_off.numel() - 1
    margin = out.get("margin")
    _check(lib().trj_argmax_accept(
        _dev(logits, name="logits"), _dtype_code(logits), vocab, _dev(tokens, torch.int32, "tokens"),
        _dev(parent, torch.int32, "parent"), _dev(depth, torch.int32, "depth"), _dev(row_off, torch.int32, "row_off"),
        batch, rows, _dev(out["node_argmax"], torch.int32), _dev(margin, torch.float32) if margin is not None else None,
        _dev(out["k_acc"], torch.int32), _dev(out["path"], torch.int32), _dev(out["bonus"], torch.int32),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)))


STATIC_MAX_ROWS = 1024


def argmax_accept_static(logits, tokens, parent, depth, row_off, out, *, stream=None) -> None:
    """trj_argmax_accept_static: the workspace-free variant of :func:`argmax_accept`.

    For hosts that may not allocate device memory (see ``include/trj.h``): the scratch is a fixed array inside
    the library, good for ``STATIC_MAX_ROWS`` rows in total.  Nothing is allocated here either: ``out`` must hold
    preallocated CUDA tensors ``node_argmax`` [rows] int32, ``margin`` [rows] float32 (or None), ``k_acc`` [B],
    ``path`` [B, PATH_STRIDE] and ``bonus`` [B] int32.  Calls share the one array, so do not let two of them run
    on the GPU at the same time; make the first call on a device outside any stream capture."""
    torch = _torch()
    rows, vocab = logits.shape
    batch = row_off.numel() - 1
    margin = out.get("margin")
    _check(lib().trj_argmax_accept_static(
        _dev(logits, name="logits"), _dtype_code(logits), vocab, _dev(tokens, torch.int32, "tokens"),
        _dev(parent, torch.int32, "parent"), _dev(depth, torch.int32, "depth"), _dev(row_off, torch.int32, "row_off"),
        batch, rows, _dev(out["node_argmax"], torch.int32), _dev(margin, torch.float32) if margin is not None else None,
        _dev(out["k_acc"], torch.int32), _dev(out["path"], torch.int32), _dev(out["bonus"], torch.int32), _stream(stream)))


def compact_rows(k_cache, v_cache, seq_len, k_acc, path, stream=None) -> None:
    """trj_compact_rows on caches [L, B, H, max_seq, D]; seq_len is advanced in place."""
    torch = _torch()
    n_layers, batch, n_heads, max_seq, hd = k_cache.shape
    _check(lib().trj_compact_rows(_dev(k_cache, name="k_cache"), _dev(v_cache, k_cache.dtype, "v_cache"), n_layers,
                                  batch, n_heads, max_seq, hd, _dtype_code(k_cache),
                                  _dev(seq_len, torch.int32, "seq_len"), _dev(k_acc, torch.int32, "k_acc"),
                                  _dev(path, torch.int32, "path"), _stream(stream)))


def gemm(x, w, *, out=None, workspace=None, stream=None):
    """trj_gemm: y [M, N] fp32 = x [M, K] . w [N, K]^T.  The first int32 of ``workspace`` is a device
    status word (0, or 4 after a bounded device-side wait expired); a fresh workspace is zeroed here."""
    torch = _torch()
    m, k = x.shape
    n = w.shape[0]
    if out is None:
        out = torch.empty(m, n, dtype=torch.float32, device=x.device)
    if workspace is None:
        workspace = _scratch(lib().trj_gemm_workspace(m, n, k), x.device, zero=True)
    _check(lib().trj_gemm(_dev(x, name="x"), _dev(w, x.dtype, "w"), _dev(out, torch.float32, "out"), m, n, k,
                          _dtype_code(x), _dev(workspace, torch.uint8), workspace.numel(), _stream(stream)))
    return out


def selftest_wait_expiry(polls: int = 256, stream=None) -> int:
    """trj_selftest_wait_expiry: returns the status word a wait that nobody satisfies leaves behind (4)."""
    torch = _torch()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(lib().trj_selftest_wait_expiry(_dev(status), int(polls), _stream(stream)))
    torch.cuda.synchronize()
    return int(status.item())


def draft_tokens(context, n_ctx, window, n_branches: int, branch_len: int, draws, stream=None):
    """trj_draft_tokens: the next tree's tokens [1 + W + R*Lr] (int32, device) from device buffers.

    context: int32 [capacity], n_ctx: int32 [1], window: int32 [W], draws: int64 [W + R*Lr], all CUDA tensors."""
    torch = _torch()
    w = int(window.numel())
    out = torch.empty(1 + w + n_branches * branch_len, dtype=torch.int32, device=context.device)
    _check(lib().trj_draft_tokens(_dev(context, torch.int32, "context"), _dev(n_ctx, torch.int32, "n_ctx"),
                                  _dev(window, torch.int32, "window") if w else None, w, n_branches, branch_len,
                                  _dev(draws, torch.int64, "draws"), _dev(out), _stream(stream)))
    return out


def commit_refill(tokens, parent, node_argmax, k_acc, path, bonus, context, n_ctx, width: int, draws, stream=None):
    """trj_commit_refill: appends the accepted tokens and the bonus to ``context`` (in place, ``n_ctx`` advanced) and
    returns (next window [width] int32, overflow flag [1] int32), both on the device."""
    torch = _torch()
    window = torch.empty(max(width, 1), dtype=torch.int32, device=context.device)
    overflow = torch.zeros(1, dtype=torch.int32, device=context.device)
    _check(lib().trj_commit_refill(_dev(tokens, torch.int32, "tokens"), _dev(parent, torch.int32, "parent"),
                                   _dev(node_argmax, torch.int32, "node_argmax"), int(tokens.numel()),
                                   _dev(k_acc, torch.int32, "k_acc"), _dev(path, torch.int32, "path"),
                                   _dev(bonus, torch.int32, "bonus"), _dev(context, torch.int32, "context"),
                                   int(context.numel()), _dev(n_ctx, torch.int32, "n_ctx"), width,
                                   _dev(draws, torch.int64, "draws"), _dev(window), _dev(overflow), _stream(stream)))
    return window[:width], overflow


class Model:
    """A decoder context (trj_create) plus its KV cache; methods map one to one onto the C ABI."""

    def __init__(self, cfg, layers: List[Dict[str, "object"]], glob: Dict[str, "object"], *,
                 max_batch: int = 1, max_seq: int = 2048, max_rows: int = MAX_ROWS):
        """``cfg`` has n_layers, d_model, n_heads, head_dim, d_ff, vocab, rms_eps, rope_theta, dtype
        ("bf16" | "f32") and optionally n_kv_heads (0 = n_heads); ``layers[l]`` and ``glob`` hold CUDA tensors
        named as in trj_weights."""
        torch = _torch()
        self.cfg = cfg
        self.tdtype = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
        self.max_batch, self.max_seq, self.max_rows = max_batch, max_seq, max_rows
        self._keep = (layers, glob)
        dev = glob["embed"].device
        self.device = dev
        self.ccfg = ModelCfg(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.head_dim, cfg.d_ff, cfg.vocab,
                             cfg.rms_eps, cfg.rope_theta, BF16 if cfg.dtype == "bf16" else F32,
                             max_batch, max_seq, max_rows, int(getattr(cfg, "n_kv_heads", 0) or 0))
        need = lib().trj_workspace_bytes(C.byref(self.ccfg))
        if need == 0:
            raise TrjError(1, lib().trj_last_error().decode())
        self.workspace = torch.zeros(need, dtype=torch.uint8, device=dev)

        def table(name, dtype):
            arr = (C.c_void_p * cfg.n_layers)()
            for l in range(cfg.n_layers):
                arr[l] = _dev(layers[l][name], dtype, name).value
            return arr
        self._tables = {n: table(n, torch.float32 if "norm" in n else self.tdtype)
                        for n in ("attn_norm", "wqkv", "wo", "mlp_norm", "w_gate_up", "w_down")}
        w = Weights(_dev(glob["embed"], self.tdtype, "embed"), _dev(glob["lm_head"], self.tdtype, "lm_head"),
                    _dev(glob["final_norm"], torch.float32, "final_norm"),
                    *(C.cast(self._tables[n], C.POINTER(C.c_void_p))
                      for n in ("attn_norm", "wqkv", "wo", "mlp_norm", "w_gate_up", "w_down")))
        self._handle = C.c_void_p()
        _check(lib().trj_create(C.byref(self.ccfg), C.byref(w), _dev(self.workspace), need, C.byref(self._handle)))
        shape = (cfg.n_layers, max_batch, int(getattr(cfg, "n_kv_heads", 0) or cfg.n_heads), max_seq, cfg.head_dim)
        self.k_cache = torch.zeros(shape, dtype=self.tdtype, device=dev)
        self.v_cache = torch.zeros(shape, dtype=self.tdtype, device=dev)
        self.seq_len = torch.zeros(max_batch, dtype=torch.int32, device=dev)

    def close(self) -> None:
        if getattr(self, "_handle", None) is not None and self._handle.value:
            lib().trj_destroy(self._handle)
            self._handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def device_status(self, clear: bool = False, stream=None) -> None:
        """trj_device_status: raises TrjError (status 4) if a bounded device-side wait has expired."""
        _check(lib().trj_device_status(self._handle, 1 if clear else 0, _stream(stream)))

    def profile_enable(self, on: bool = True) -> None:
        _check(lib().trj_profile_enable(self._handle, 1 if on else 0))

    def profile_read(self, keep: bool = False) -> Dict[str, Tuple[float, int]]:
        """trj_profile_read: {category: (device ms, launches)} since the last read (kept if ``keep``)."""
        ms = (C.c_float * len(PROF_CATEGORIES))()
        n = (C.c_int32 * len(PROF_CATEGORIES))()
        _check(lib().trj_profile_read(self._handle, ms, n, 1 if keep else 0))
        return {c: (float(ms[i]), int(n[i])) for i, c in enumerate(PROF_CATEGORIES)}

    def prefill(self, tokens, b: int = 0, stream=None):
        """trj_prefill: returns the device tensor holding the first greedy token."""
        torch = _torch()
        first = torch.empty(1, dtype=torch.int32, device=self.device)
        _check(lib().trj_prefill(self._handle, _dev(self.k_cache), _dev(self.v_cache), _dev(self.seq_len), b,
                                 _dev(tokens, torch.int32, "tokens"), tokens.numel(), _dev(first), _stream(stream)))
        return first

    def verify_step(self, tokens, parent, depth, anc, row_off, *, max_rows: int, max_len: int,
                    want_logits: bool = False, want_margin: bool = False, node_argmax=None, stream=None):
        """trj_verify_step: dict(node_argmax, margin | None, logits | None).  ``node_argmax`` may be a
        preallocated int32 tensor [rows]."""
        torch = _torch()
        rows, batch = tokens.numel(), row_off.numel() - 1
        if node_argmax is None:
            node_argmax = torch.empty(rows, dtype=torch.int32, device=self.device)
        margin = torch.empty(rows, dtype=torch.float32, device=self.device) if want_margin else None
        logits = torch.empty(rows, self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        _check(lib().trj_verify_step(
            self._handle, _dev(self.k_cache), _dev(self.v_cache), _dev(self.seq_len),
            _dev(tokens, torch.int32, "tokens"), _dev(parent, torch.int32, "parent"), _dev(depth, torch.int32, "depth"),
            _dev(anc, torch.int64, "anc"), anc.shape[1], _dev(row_off, torch.int32, "row_off"), batch, rows,
            max_rows, max_len, _dev(node_argmax), _dev(margin) if want_margin else None,
            _dev(logits) if want_logits else None, _stream(stream)))
        return {"node_argmax": node_argmax, "margin": margin, "logits": logits}

    # ---- tensor-parallel stepping: this context is one rank's slice of the decoder
    def tp_segments(self) -> int:
        return int(lib().trj_tp_segments(self._handle))

    def tp_begin(self, tokens, parent, depth, anc, row_off, *, max_rows: int, max_len: int, stream=None) -> None:
        """trj_tp_begin: the tensors must stay alive until tp_finish (kept on the object)."""
        torch = _torch()
        self._tp_keep = (tokens, parent, depth, anc, row_off)
        _check(lib().trj_tp_begin(
            self._handle, _dev(self.k_cache), _dev(self.v_cache), _dev(self.seq_len),
            _dev(tokens, torch.int32, "tokens"), _dev(parent, torch.int32, "parent"), _dev(depth, torch.int32, "depth"),
            _dev(anc, torch.int64, "anc"), anc.shape[1], _dev(row_off, torch.int32, "row_off"), row_off.numel() - 1,
            tokens.numel(), max_rows, max_len, _stream(stream)))

    def tp_segment(self, segment: int, stream=None) -> None:
        _check(lib().trj_tp_segment(self._handle, int(segment), _stream(stream)))

    def tp_exchange_tensor(self):
        """trj_tp_exchange_buffer as a float32 tensor [rows, d_model] that aliases the workspace (no copy)."""
        torch = _torch()
        ptr, count = _VP(), _SZ()
        _check(lib().trj_tp_exchange_buffer(self._handle, C.byref(ptr), C.byref(count)))
        off = ptr.value - self.workspace.data_ptr()
        if off < 0 or off + 4 * count.value > self.workspace.numel():
            raise TrjError(1, "exchange buffer outside the workspace")
        return self.workspace[off:off + 4 * count.value].view(torch.float32).view(-1, self.cfg.d_model)

    def tp_finish(self, *, want_logits: bool = False, want_margin: bool = False, stream=None):
        """trj_tp_finish: dict(node_argmax, margin | None, logits | None) as verify_step."""
        torch = _torch()
        rows = self._tp_keep[0].numel()
        node_argmax = torch.empty(rows, dtype=torch.int32, device=self.device)
        margin = torch.empty(rows, dtype=torch.float32, device=self.device) if want_margin else None
        logits = torch.empty(rows, self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        _check(lib().trj_tp_finish(self._handle, _dev(node_argmax), _dev(margin) if want_margin else None,
                                   _dev(logits) if want_logits else None, _stream(stream)))
        return {"node_argmax": node_argmax, "margin": margin, "logits": logits}

    def node_topk(self, rows: int, k: int, out=None, stream=None):
        """trj_node_topk: [rows, k] int32 ids of the k largest logits of every row of the latest verify_step."""
        torch = _torch()
        if out is None:
            out = torch.empty(rows, k, dtype=torch.int32, device=self.device)
        _check(lib().trj_node_topk(self._handle, int(rows), int(k), _dev(out, torch.int32, "topk"), _stream(stream)))
        return out

    def accept(self, tokens, parent, depth, row_off, node_argmax, out=None, stream=None):
        """trj_accept: dict(k_acc [B], path [B, PATH_STRIDE], bonus [B]); ``out`` may hold preallocated ones."""
        torch = _torch()
        batch = row_off.numel() - 1
        i32 = dict(dtype=torch.int32, device=self.device)
        if out is not None:
            k_acc, bonus, path = out["k_acc"], out["bonus"], out["path"]
        else:
            k_acc, bonus, path = torch.empty(batch, **i32), torch.empty(batch, **i32), torch.empty(batch, PATH_STRIDE, **i32)
        _check(lib().trj_accept(self._handle, _dev(tokens, torch.int32), _dev(parent, torch.int32),
                                _dev(depth, torch.int32), _dev(row_off, torch.int32), batch, tokens.numel(),
                                _dev(node_argmax, torch.int32), _dev(k_acc), _dev(path), _dev(bonus), _stream(stream)))
        return {"k_acc": k_acc, "path": path, "bonus": bonus}

    def compact_kv(self, k_acc, path, batch: int = 1, stream=None) -> None:
        """trj_compact_kv: moves the accepted rows and advances seq_len."""
        torch = _torch()
        _check(lib().trj_compact_kv(self._handle, _dev(self.k_cache), _dev(self.v_cache), _dev(self.seq_len), batch,
                                    _dev(k_acc, torch.int32), _dev(path, torch.int32), _stream(stream)))

    def decode_device(self, context, n_ctx, n_ctx_now: int, window, n_branches: int, branch_len: int, draws,
                      n_steps: int, k_log=None, stream=None) -> None:
        """trj_decode_device: ``n_steps`` decode steps of sequence 0 without the host in between (nothing is
        synchronised).  context int32 [capacity], n_ctx int32 [1], window int32 [W], draws int64
        [n_steps, W + R*Lr], k_log int32 [n_steps] or None: CUDA tensors, updated in place."""
        torch = _torch()
        w = int(window.numel())
        _check(lib().trj_decode_device(self._handle, _dev(self.k_cache), _dev(self.v_cache), _dev(self.seq_len),
                                       _dev(context, torch.int32, "context"), int(context.numel()),
                                       _dev(n_ctx, torch.int32, "n_ctx"), int(n_ctx_now),
                                       _dev(window, torch.int32, "window") if w else None, w, n_branches, branch_len,
                                       _dev(draws, torch.int64, "draws"), int(n_steps),
                                       _dev(k_log, torch.int32, "k_log") if k_log is not None else None, _stream(stream)))

    def decode_device_tree(self, context, n_ctx, n_ctx_now: int, parent, rank, top_k: int, n_retrieved: int, drafts,
                           draws, n_steps: int, k_log=None, stream=None) -> None:
        """trj_decode_device_tree: ``n_steps`` decode steps of sequence 0 over a static tree template with top-K
        siblings, without the host in between.  parent / rank: host int arrays [M]; context int32 [capacity], n_ctx
        int32 [1], drafts int32 [M - 1], draws int64 [n_steps, M - 1 + n_retrieved], k_log int32 [n_steps] or None:
        CUDA tensors, updated in place."""
        torch = _torch()
        parent, rank = _i32(parent), _i32(rank)
        _check(lib().trj_decode_device_tree(
            self._handle, _dev(self.k_cache), _dev(self.v_cache), _dev(self.seq_len),
            _dev(context, torch.int32, "context"), int(context.numel()), _dev(n_ctx, torch.int32, "n_ctx"), int(n_ctx_now),
            _p32(parent), _p32(rank), len(parent), int(top_k), int(n_retrieved),
            _dev(drafts, torch.int32, "drafts") if len(parent) > 1 else None, _dev(draws, torch.int64, "draws"), int(n_steps),
            _dev(k_log, torch.int32, "k_log") if k_log is not None else None, _stream(stream)))

    def set_draft_source(self, stream=None, take=None) -> None:
        """trj_set_draft_source: ``stream`` int32 [n] guesses by context position, ``take`` int32 [n_steps] how many
        of them each step of the next decode_device call plants into branch 0 (CUDA tensors, kept alive here);
        ``None`` removes the source."""
        torch = _torch()
        self._draft_src = (stream, take)
        if stream is None:
            _check(lib().trj_set_draft_source(self._handle, None, 0, None, 0))
        else:
            _check(lib().trj_set_draft_source(self._handle, _dev(stream, torch.int32, "stream"), int(stream.numel()),
                                              _dev(take, torch.int32, "take"), int(take.numel())))

    def step_host(self, root: int, window, branches, max_len: int, stream=None) -> Dict[str, object]:
        """trj_step_host: one whole decode step from host integers; returns host results."""
        window = _i32(window).reshape(-1)
        br = _i32(branches)
        br = br.reshape(br.shape[0], -1) if br.size else np.zeros((0, 0), np.int32)
        r, bl = (br.shape[0], br.shape[1]) if br.size else (0, 0)
        hb = self._step_host_buffers()                       # marshalling state that does not change between calls
        tokens, parent, pred, path = hb["tokens"], hb["parent"], hb["pred"], hb["path"]
        n, k, bonus = hb["n"], hb["k"], hb["bonus"]
        _check(hb["fn"](self._handle, hb["kc"], hb["vc"], hb["len"], max_len,
                        int(root), _p32(window), len(window), _p32(br), r, bl, hb["p_tokens"], hb["p_parent"],
                        hb["r_n"], hb["p_pred"], hb["r_k"], hb["p_path"], hb["r_bonus"], _stream(stream)))
        m = n.value
        return {"tokens": tokens[:m].copy(), "parent": parent[:m].copy(), "node_argmax": pred[:m].copy(), "k_acc": k.value,
                "path": path[:k.value + 1].copy(), "bonus": bonus.value}

    def _step_host_buffers(self):
        hb = getattr(self, "_hb", None)
        if hb is None or hb["ptrs"] != (self.k_cache.data_ptr(), self.v_cache.data_ptr(), self.seq_len.data_ptr()):
            tokens, parent, pred = (np.zeros(MAX_ROWS, np.int32) for _ in range(3))
            path = np.zeros(PATH_STRIDE, np.int32)
            n, k, bonus = C.c_int32(0), C.c_int32(0), C.c_int32(0)
            hb = {"ptrs": (self.k_cache.data_ptr(), self.v_cache.data_ptr(), self.seq_len.data_ptr()),
                  "fn": lib().trj_step_host, "kc": _dev(self.k_cache), "vc": _dev(self.v_cache), "len": _dev(self.seq_len),
                  "tokens": tokens, "parent": parent, "pred": pred, "path": path, "n": n, "k": k, "bonus": bonus,
                  "p_tokens": _p32(tokens), "p_parent": _p32(parent), "p_pred": _p32(pred), "p_path": _p32(path),
                  "r_n": C.byref(n), "r_k": C.byref(k), "r_bonus": C.byref(bonus)}
            self._hb = hb
        return hb
