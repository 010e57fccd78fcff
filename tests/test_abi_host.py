"""CPU-only checks of the boundary: exported symbols, host-side integer entry points, argument errors."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    with open(os.path.join(ROOT, "include", "trj.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(trj_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(trj):
    names = declared_symbols()
    assert len(names) >= 20
    handle = ctypes.CDLL(trj.LIB_PATH)
    for n in names:
        assert hasattr(handle, n), f"{n} is declared in trj.h but not exported"
    assert sorted(trj.EXPORTS) == names
    assert "sm_100a" in trj.version()


def test_build_tree_matches_oracle(trj):
    for seed, (w, r, bl) in enumerate([(4, 2, 3), (5, 9, 3), (0, 0, 0), (1, 0, 0), (0, 3, 2), (60, 1, 5), (100, 9, 3)]):
        g = synth.stream(seed, "bt")
        root = int(g.integers(0, 1000))
        window = g.integers(0, 1000, size=w)
        branches = g.integers(0, 1000, size=(r, bl))
        got = trj.build_tree(root, window, branches)
        tokens, parent = oracle.build_tree(root, window, branches)
        np.testing.assert_array_equal(got["tokens"], tokens)
        np.testing.assert_array_equal(got["parent"], parent)
        np.testing.assert_array_equal(got["depth"], oracle.depths(parent))
        want = oracle.pack_mask(oracle.ancestor_mask(parent))
        np.testing.assert_array_equal(got["anc"][:, :want.shape[1]], want)
        assert not got["anc"][:, want.shape[1]:].any()


def test_tree_from_parents_matches_oracle_on_random_trees(trj):
    for seed, m in enumerate([1, 2, 10, 63, 64, 65, 127, 128]):
        parent = synth.random_tree(seed, m, min(8, max(1, m - 1)), 3) if m > 1 else np.array([-1], np.int32)
        depth, anc = trj.tree_from_parents(parent)
        np.testing.assert_array_equal(depth, oracle.depths(parent))
        want = oracle.pack_mask(oracle.ancestor_mask(parent))
        np.testing.assert_array_equal(anc[:, :want.shape[1]], want)
    depth, anc = trj.tree_from_parents(synth.chain_parents(128))
    assert depth[127] == 127 and int(anc[127, 0]) == 2 ** 64 - 1 and int(anc[127, 1]) == 2 ** 64 - 1


def test_tree_errors(trj):
    with pytest.raises(trj.TrjError) as e:
        trj.tree_from_parents([-1, 1])
    assert e.value.status == 1 and "parent[1]" in str(e.value)
    with pytest.raises(trj.TrjError) as e:
        trj.tree_from_parents([0, 0])
    assert e.value.status == 1
    with pytest.raises(trj.TrjError) as e:
        trj.tree_from_parents(synth.chain_parents(129), anc_words=3)
    assert e.value.status == 2
    with pytest.raises(trj.TrjError) as e:
        trj.tree_from_parents(synth.chain_parents(65), anc_words=1)
    assert e.value.status == 2
    with pytest.raises(trj.TrjError) as e:
        trj.build_tree(1, [1] * 5, np.ones((9, 3), np.int32), max_rows=32)      # 33 rows
    assert e.value.status == 2
    with pytest.raises(trj.TrjError) as e:
        trj.build_tree(1, [1] * 5, [], max_rows=200)
    assert e.value.status == 2


def test_retrieve_and_refill_match_oracle(trj):
    for seed in range(40):
        g = synth.stream(seed, "ctx")
        n = int(g.integers(1, 60))
        vocab = int(g.integers(2, 6))                       # tiny vocabulary: many repeated n-grams
        ctx = g.integers(0, vocab, size=n).astype(np.int32)
        r, bl = int(g.integers(0, 5)), int(g.integers(1, 6))
        draws = synth.noise_draws(seed, 1, r * bl + 8)
        got = trj.retrieve(ctx, r, bl, draws)
        want = oracle.retrieve(list(ctx), r, bl, draws)
        assert got.tolist() == want, (seed, ctx.tolist())
        m = int(g.integers(1, 30))
        parent = synth.random_tree(seed, m, 6, 3, name="rf") if m > 1 else np.array([-1], np.int32)
        pred = g.integers(0, 100, size=m).astype(np.int32)
        best = int(g.integers(0, m))
        w = int(g.integers(0, 8))
        got_w = trj.refill_window(parent, pred, best, w, ctx, draws)
        assert got_w.tolist() == oracle.refill_window(parent, pred, best, w, list(ctx), draws)


def test_device_entry_points_reject_bad_arguments_before_any_launch(trj):
    """Null pointers and bad shapes are refused on the host: no CUDA call is reached, so this runs without a GPU."""
    lib = trj.lib()
    nul = None
    assert lib.trj_tree_attention(nul, nul, nul, nul, nul, nul, 1, 1, 1, 1, 1, 128, 16, 16, 1, nul, nul, 0, nul) == 1
    assert "null" in lib.trj_last_error().decode()
    assert lib.trj_argmax_accept(nul, 1, 10, nul, nul, nul, nul, 1, 1, nul, nul, nul, nul, nul, nul, 0, nul) == 1
    assert lib.trj_compact_rows(nul, nul, 1, 1, 1, 1, 128, 1, nul, nul, nul, nul) == 1
    assert lib.trj_gemm(nul, nul, nul, 1, 1, 1, 1, nul, 0, nul) == 1
    fake = ctypes.c_void_p(256)                              # never dereferenced: checks fail first
    assert lib.trj_tree_attention(fake, fake, fake, fake, fake, fake, 1, 1, 1, 1, 1, 96, 16, 16, 1, fake, fake, 256, nul) == 5
    assert lib.trj_tree_attention(fake, fake, fake, fake, fake, fake, 1, 1, 1, 200, 1, 128, 16, 16, 1, fake, fake, 256, nul) == 2
    assert lib.trj_tree_attention(fake, fake, fake, fake, fake, fake, 1, 1, 1, 70, 1, 128, 16, 16, 1, fake, fake, 256, nul) == 1
    assert lib.trj_tree_attention(fake, fake, fake, fake, fake, fake, 1, 1, 1, 8, 1, 128, 16, 32, 1, fake, fake, 256, nul) == 2
    assert lib.trj_tree_attention(fake, fake, fake, fake, fake, fake, 1, 1, 1, 8, 1, 128, 16, 16, 7, fake, fake, 256, nul) == 1
    assert lib.trj_argmax_accept(fake, 1, 10, fake, fake, fake, fake, 100, 100, fake, nul, fake, fake, fake, fake, 1 << 20, nul) == 2
    # device-side drafting / commit / decode loop: pointers and sizes are checked before anything is launched
    assert lib.trj_draft_tokens(nul, nul, nul, 4, 2, 3, nul, nul, nul) == 1
    assert lib.trj_draft_tokens(fake, fake, fake, 4, 65, 1, fake, fake, nul) == 2          # more than 64 branches
    assert lib.trj_draft_tokens(fake, fake, fake, 100, 10, 3, fake, fake, nul) == 2        # 131 rows
    assert lib.trj_draft_tokens(fake, fake, nul, 4, 2, 3, fake, fake, nul) == 1            # window missing
    assert lib.trj_commit_refill(nul, nul, nul, 4, nul, nul, nul, nul, 10, nul, 2, nul, nul, nul, nul) == 1
    assert lib.trj_commit_refill(fake, fake, fake, 500, fake, fake, fake, fake, 10, fake, 2, fake, fake, nul, nul) == 2
    assert lib.trj_decode_device(nul, fake, fake, fake, fake, 10, fake, 1, fake, 4, 2, 3, fake, 1, nul, nul) == 1
    i32p = lambda a: np.asarray(a, np.int32).ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    assert lib.trj_decode_device_tree(nul, fake, fake, fake, fake, 10, fake, 1, i32p([-1, 0]), i32p([0, 0]), 2, 1, 0, fake, fake, 1, nul, nul) == 1
    # the step of a rank that holds a slice of the weights: no context, no step
    assert lib.trj_tp_segments(nul) == 0
    assert lib.trj_tp_begin(nul, fake, fake, fake, fake, fake, fake, fake, 2, fake, 1, 1, 1, 1, nul) == 1
    assert lib.trj_tp_segment(nul, 0, nul) == 1
    assert lib.trj_tp_exchange_buffer(nul, nul, nul) == 1
    assert lib.trj_tp_finish(nul, fake, nul, nul, nul) == 1
    cfg = trj.ModelCfg(2, 256, 4, 48, 688, 1024, 1e-5, 1e4, 0, 1, 256, 16)
    assert lib.trj_workspace_bytes(ctypes.byref(cfg)) == 0
    cfg = trj.ModelCfg(2, 256, 4, 64, 688, 1024, 1e-5, 1e4, 0, 1, 256, 300)
    assert lib.trj_workspace_bytes(ctypes.byref(cfg)) == 0
    cfg = trj.ModelCfg(2, 256, 4, 64, 688, 1024, 1e-5, 1e4, 0, 1, 256, 16)
    assert lib.trj_workspace_bytes(ctypes.byref(cfg)) > 0
    out = ctypes.c_void_p()
    assert lib.trj_create(ctypes.byref(cfg), None, fake, 1 << 30, ctypes.byref(out)) == 1
    assert lib.trj_destroy(None) == 0


def test_refill_tree_matches_oracle(trj):
    """trj_refill_tree against the oracle on seeded templates, every possible winner, random top-K tables."""
    for seed, (n_nodes, n_retr, k) in enumerate([(63, 5, 10), (20, 0, 5), (12, 3, 6), (0, 2, 1)]):
        parent, rank = synth.tree_template(seed, n_nodes, 4, 10, n_retr)
        m = len(parent)
        g = synth.stream(seed, "refill_tree")
        topk = g.integers(0, 5000, size=(m, k)).astype(np.int32)
        context = g.integers(0, 5000, size=37).astype(np.int32)
        retrieved = g.integers(0, 5000, size=n_retr).astype(np.int32)
        for best in range(m):
            draws = g.integers(0, 2 ** 31 - 1, size=max(m - 1, 1))
            want = oracle.refill_tree(parent, rank, topk, best, context, draws, retrieved)
            got = trj.refill_tree(parent, rank, topk, best, context, draws, retrieved)
            assert got.tolist() == want
    # chain + ranks 0 = the Jacobi window refill
    chain = synth.chain_parents(7)
    pred = np.arange(7, dtype=np.int32) + 50
    got = trj.refill_tree(chain, np.zeros(7, np.int32), pred[:, None], 2, [1, 2, 3], np.zeros(6, np.int64))
    assert got.tolist()[:4] == trj.refill_window(chain, pred, 2, 4, [1, 2, 3], np.zeros(4, np.int64)).tolist()
    with pytest.raises(trj.TrjError):
        trj.refill_tree([-1, 0], [0, 3], np.zeros((2, 2), np.int32), 0, [1], [0])       # rank 3 with K = 2


def test_default_build_has_no_clock_stamps(trj):
    """The timeline entry points exist in every build but only the -DTRJ_TIMELINE build records anything."""
    with pytest.raises(trj.TrjError) as e:
        trj.timeline_read(4)
    assert e.value.status == 5
