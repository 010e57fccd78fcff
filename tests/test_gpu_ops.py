"""GPU parity of the op-level entry points against the CPU oracle, through the C ABI.

Tolerances: attention outputs max |err| <= 2e-2 for bf16 storage (the bound the task states) and
<= 2e-5 for fp32 storage (fp32 accumulation over a few thousand terms of O(1) values); integer
results (arg-max, k, path, bonus, sequence lengths) and compacted cache bytes are bit-exact.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import AttnCase, anc_dev, i32, to_dev

pytestmark = pytest.mark.gpu
TOL = {"bf16": 2e-2, "f32": 2e-5}


def check_attention(trj, case, heads=None, seqs=None):
    need = trj.tree_attention_workspace(int(case.row_off_host[-1]), len(case.rows), case.h, case.d, case.max_len)
    ws = torch.zeros(max(256, need), dtype=torch.uint8, device="cuda")
    out = case.run(trj, workspace=ws).float().cpu().numpy()
    torch.cuda.synchronize()
    assert int(ws[:4].view(torch.int32)[0]) == 0           # no device-side wait expired
    worst = 0.0
    for b in (range(len(case.rows)) if seqs is None else seqs):
        r0, r1 = case.row_off_host[b], case.row_off_host[b + 1]
        ref = case.oracle_rows(oracle, b, heads)
        hs = list(range(case.h)) if heads is None else list(heads)
        err = np.abs(out[r0:r1][:, hs] - ref).max()
        worst = max(worst, err)
    assert np.isfinite(out).all()
    assert worst <= TOL[case.dtype], worst
    return worst


@pytest.mark.parametrize("dtype,h,d,s,m", [
    ("bf16", 4, 128, 300, 37), ("bf16", 2, 128, 0, 9), ("bf16", 2, 128, 1, 1), ("bf16", 2, 128, 127, 64),
    ("bf16", 2, 128, 128, 65), ("bf16", 2, 128, 129, 128), ("bf16", 3, 128, 515, 33),
    ("f32", 4, 64, 70, 11), ("f32", 2, 64, 0, 1), ("f32", 2, 128, 200, 70), ("bf16", 2, 64, 260, 40),
])
def test_tree_attention_small(trj, dtype, h, d, s, m):
    parent = synth.random_tree(s + m, m, min(8, m - 1), 3) if m > 1 else np.array([-1], np.int32)
    case = AttnCase(trj, 1, h, d, [s], [m], [parent], dtype, pad=3)
    check_attention(trj, case)


@pytest.mark.parametrize("h,s,m", [
    (2, 3000, 128),      # clusters of 4 with six or seven key tiles per CTA (the K/V ring wraps)
    (40, 700, 20),       # 4 x 40 CTAs would not fit: clusters of 2
    (80, 1500, 16),      # no clusters and more tiles than one CTA takes per head: contiguous ranges + merge kernel
    (80, 600, 16),       # no clusters, few tiles: one CTA per head
])
def test_tree_attention_launch_shapes_single_sequence(trj, h, s, m):
    """One sequence, head counts and lengths that exercise every launch shape the host chooses from."""
    case = AttnCase(trj, h, h, 128, [s], [m], [synth.random_tree(h + s, m, min(8, m - 1), 3)], "bf16", pad=5)
    check_attention(trj, case, heads=[0, h // 2, h - 1])


def test_tree_attention_chain_is_causal(trj):
    """A chain tree on the GPU reproduces causal attention (oracle pinned to a library routine)."""
    m = 96
    case = AttnCase(trj, 2, 2, 128, [40], [m], [synth.chain_parents(m)], "bf16")
    check_attention(trj, case)


def test_tree_attention_is_deterministic(trj):
    case = AttnCase(trj, 3, 4, 128, [777], [48], [synth.random_tree(3, 48, 6, 3)], "bf16")
    a, b = case.run(trj), case.run(trj)
    assert torch.equal(a, b)


def test_tree_attention_config2_full(trj):
    """32 heads x 128, prefix 1024, 64-row tree of depth 6 with 1-3 children."""
    case = AttnCase(trj, 1, 32, 128, [1024], [64], [synth.random_tree(1, 64, 6, 3)], "bf16")
    check_attention(trj, case)


def test_tree_attention_config4_full(trj):
    """32 heads x 128, prefix 8192, 128-row tree of depth 8; every head is compared."""
    case = AttnCase(trj, 3, 32, 128, [8192], [128], [synth.random_tree(3, 128, 8, 4)], "bf16", pad=7)
    check_attention(trj, case)


def test_tree_attention_config5_ragged_batch(trj):
    s, m = synth.ragged_batch(4, 8, (256, 4096), (16, 64))
    parents = [synth.random_tree(40 + i, int(mi), 6, 3) for i, mi in enumerate(m)]
    case = AttnCase(trj, 4, 32, 128, s.tolist(), m.tolist(), parents, "bf16", max_seq=4096 + 64)
    check_attention(trj, case, heads=[0, 1, 7, 12, 16, 23, 30, 31])


@pytest.mark.parametrize("dtype,h,hk,d,prefixes,rows", [
    ("bf16", 32, 8, 128, [1024], [64]),                    # LLaMA-3 head layout on the config-2 shape (clusters)
    ("bf16", 8, 2, 128, [3000], [128]),                    # long prefix: clusters whose ring wraps
    ("bf16", 32, 8, 128, [700, 2200, 256], [33, 16, 64]),  # ragged batch: contiguous ranges + merge kernel
    ("bf16", 4, 1, 128, [130], [9]),                       # multi-query
    ("f32", 4, 2, 64, [70], [11]),                         # the generic kernel
])
def test_tree_attention_grouped_query(trj, dtype, h, hk, d, prefixes, rows):
    """Grouped-query attention (LLaMA-3 family, Table 2): H query heads over Hkv K/V heads."""
    parents = [synth.random_tree(70 + i, m, min(6, m - 1), 3) for i, m in enumerate(rows)]
    case = AttnCase(trj, 9, h, d, prefixes, rows, parents, dtype, pad=4, kv_heads=hk)
    heads = None if h <= 8 else [0, 3, 4, 7, 13, 20, 27, 31]
    check_attention(trj, case, heads=heads)


def test_tensor_core_shapes_are_never_rerouted(trj):
    """A bf16 / head_dim-128 attention call or a projection of a tensor-core shape with a short or misaligned
    workspace is an error, not a silent run on the generic kernel."""
    case = AttnCase(trj, 5, 2, 128, [100], [9], [synth.random_tree(5, 9, 4, 3)], "bf16")
    need = trj.tree_attention_workspace(9, 1, 2, 128, 109)
    with pytest.raises(trj.TrjError) as e:
        case.run(trj, workspace=torch.zeros(need - 256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 2
    with pytest.raises(trj.TrjError) as e:
        case.run(trj, workspace=torch.zeros(need + 512, dtype=torch.uint8, device="cuda")[16:])
    assert e.value.status == 1
    x = torch.zeros(8, 256, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(64, 256, dtype=torch.bfloat16, device="cuda")
    gneed = trj.lib().trj_gemm_workspace(8, 64, 256)
    with pytest.raises(trj.TrjError) as e:
        trj.gemm(x, w, workspace=torch.zeros(gneed + 512, dtype=torch.uint8, device="cuda")[16:])
    assert e.value.status == 1


def test_an_expired_wait_is_reported_and_the_kernel_returns(trj):
    """The bounded wait of the tensor-core kernels, made to run out on a barrier nobody arrives at: the status
    word reads TRJ_ETIMEOUT, the launch completes by itself and the device stays usable."""
    for polls in (40, 1000):
        assert trj.selftest_wait_expiry(polls) == 4
    case = AttnCase(trj, 6, 2, 128, [200], [17], [synth.random_tree(6, 17, 4, 3)], "bf16")
    check_attention(trj, case)                             # the context still works


# ----------------------------------------------------------------------------- arg-max + acceptance
def accept_case(seed, rows_list, vocab, dtype, depth_cap=6):
    parents = [synth.random_tree(seed * 100 + i, m, min(depth_cap, max(1, m - 1)), 3) if m > 1 else np.array([-1], np.int32)
               for i, m in enumerate(rows_list)]
    logits = synth.logits(seed, sum(rows_list), vocab, dtype)
    pred = oracle.node_argmax(logits)
    off = np.concatenate([[0], np.cumsum(rows_list)]).astype(np.int32)
    tokens = np.concatenate([synth.planted_tokens(seed, p, pred[off[i]:off[i + 1]], vocab, name=f"plant{i}")
                             for i, p in enumerate(parents)])
    return parents, logits, pred, off, tokens


def check_argmax_accept(trj, seed, rows_list, vocab, dtype):
    parents, logits, pred, off, tokens = accept_case(seed, rows_list, vocab, dtype)
    depth = np.concatenate([oracle.depths(p) for p in parents])
    res = trj.argmax_accept(to_dev(logits, dtype), i32(tokens), i32(np.concatenate(parents)), i32(depth), i32(off))
    torch.cuda.synchronize()
    np.testing.assert_array_equal(res["node_argmax"].cpu().numpy(), pred)
    np.testing.assert_allclose(res["margin"].cpu().numpy(), oracle.top2_margin(logits), rtol=0, atol=1e-6)
    ks = []
    for b, p in enumerate(parents):
        k, path, bonus = oracle.accept_path(tokens[off[b]:off[b + 1]], p, pred[off[b]:off[b + 1]])
        assert int(res["k_acc"][b]) == k
        assert res["path"][b, :k + 1].tolist() == path
        assert (res["path"][b, k + 1:] == -1).all()
        assert int(res["bonus"][b]) == bonus
        ks.append(k)
    return ks


def test_argmax_accept_config2(trj):
    ks = check_argmax_accept(trj, 1, [64], 32000, "bf16")
    check_argmax_accept(trj, 2, [64], 32000, "f32")
    assert ks[0] >= 1                                      # the planted drafts make some path non-trivial


def test_argmax_accept_config5_batch(trj):
    _, m = synth.ragged_batch(4, 8, (256, 4096), (16, 64))
    ks = check_argmax_accept(trj, 4, m.tolist(), 32000, "bf16")
    assert len(set(ks)) > 1


@pytest.mark.parametrize("rows_list,vocab", [([1], 7), ([1, 1, 1], 1001), ([128], 513), ([5, 128, 2], 32000), ([64] * 64, 100)])
def test_argmax_accept_edges(trj, rows_list, vocab):
    check_argmax_accept(trj, 7, rows_list, vocab, "bf16")
    check_argmax_accept(trj, 8, rows_list, vocab, "f32")


@pytest.mark.parametrize("rows_list,vocab,k,dtype", [
    ([69], 32000, 10, "f32"), ([64], 32000, 10, "bf16"), ([33], 128256, 4, "f32"), ([1], 11, 10, "f32"),
    ([5, 128, 2], 4099, 3, "bf16"), ([16] * 8, 1001, 2, "f32"), ([7], 513, 1, "bf16"),
])
def test_topk_accept_against_oracle(trj, rows_list, vocab, k, dtype):
    """Per-row top-K (Appendix B) bit-exact against the oracle, exact ties included (bf16 logits tie often), and the
    acceptance results next to it."""
    parents, logits, pred, off, tokens = accept_case(11, rows_list, vocab, dtype)
    depth = np.concatenate([oracle.depths(p) for p in parents])
    ws = torch.zeros(trj.lib().trj_topk_accept_workspace(), dtype=torch.uint8, device="cuda")
    for _ in range(2):                                     # the workspace is left ready for the next call
        res = trj.topk_accept(to_dev(logits, dtype), i32(tokens), i32(np.concatenate(parents)), i32(depth), i32(off), k, workspace=ws)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(res["topk"].cpu().numpy(), oracle.node_topk(logits, k))
        np.testing.assert_array_equal(res["node_argmax"].cpu().numpy(), pred)
        if vocab > 1:
            np.testing.assert_allclose(res["margin"].cpu().numpy(), oracle.top2_margin(logits), rtol=0, atol=1e-6)
        for b, p in enumerate(parents):
            kk, path, bonus = oracle.accept_path(tokens[off[b]:off[b + 1]], p, pred[off[b]:off[b + 1]])
            assert int(res["k_acc"][b]) == kk and int(res["bonus"][b]) == bonus
            assert res["path"][b, :kk + 1].tolist() == path and (res["path"][b, kk + 1:] == -1).all()


@pytest.mark.parametrize("vocab,k", [(40000, 10), (128256, 7), (5000, 10)])
def test_topk_with_thousands_of_equal_values(trj, vocab, k):
    """Rows in which far more entries tie for the top than any candidate buffer holds (all equal; a plateau of 3 000
    maxima; a few distinct values above a plateau; plateaus that straddle the 32 768-entry chunks): the K smallest ids
    of the best values must come out, bit for bit as the oracle's total order (value first, then the smaller id)."""
    g = synth.stream(vocab, "plateau")
    rows = 6
    logits = g.standard_normal((rows, vocab)).astype(np.float32)
    logits[0, :] = 0.25                                                  # everything ties
    top = g.choice(vocab, size=min(3000, vocab // 2), replace=False)
    logits[1, top] = 9.0                                                 # a plateau of maxima
    logits[2, top] = 9.0; logits[2, top[:3]] = [11.0, 10.0, 10.0]        # three above it, two of them tied
    logits[3, -1500:] = 7.0; logits[3, :20] = 7.0                        # plateau at both ends of the row
    logits[4, 32768 - 600:min(vocab, 32768 + 600)] = 8.0                 # plateau across a chunk boundary
    parents = [synth.chain_parents(rows)]
    tokens = synth.prompt(3, rows, vocab)
    depth = np.concatenate([oracle.depths(p) for p in parents])
    res = trj.topk_accept(to_dev(logits, "f32"), i32(tokens), i32(np.concatenate(parents)), i32(depth), i32([0, rows]), k)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(res["topk"].cpu().numpy(), oracle.node_topk(logits, k))
    np.testing.assert_array_equal(res["node_argmax"].cpu().numpy(), oracle.node_argmax(logits))
    np.testing.assert_array_equal(res["margin"].cpu().numpy(), oracle.top2_margin(logits).astype(np.float32))


def test_argmax_ties_go_to_the_smallest_id_and_workspace_is_reusable(trj):
    rows, vocab = 9, 4099
    logits = np.zeros((rows, vocab), np.float32)
    logits[1, 4098] = 1.0; logits[1, 17] = 1.0            # tie between a late and an early id
    logits[2, :] = -3.0; logits[2, 4000] = -3.0           # all equal
    logits[3, 0] = 5.0; logits[3, 4098] = 5.0
    parent = synth.chain_parents(rows)
    depth = oracle.depths(parent)
    tokens = np.zeros(rows, np.int32)
    ws = torch.zeros(trj.argmax_accept_workspace(rows, 1), dtype=torch.uint8, device="cuda")
    for _ in range(3):                                     # the same workspace, call after call
        res = trj.argmax_accept(to_dev(logits, "f32"), i32(tokens), i32(parent), i32(depth), i32([0, rows]), workspace=ws)
        assert res["node_argmax"].tolist() == [0, 17, 0, 0, 0, 0, 0, 0, 0]
        assert res["margin"].tolist() == [0.0] * rows
        assert int(res["k_acc"][0]) == 1 and int(res["bonus"][0]) == 17      # token 0 == argmax(root) == 0, then 0 != 17


# ----------------------------------------------------------------------------- KV compaction
def check_compaction(trj, seed, n_layers, h, d, dtype, prefixes, parents, ks, max_seq):
    b = len(prefixes)
    g = synth.stream(seed, "cache")
    shape = (n_layers, b, h, max_seq, d)
    k_host = synth.round_bf16(g.standard_normal(shape, dtype=np.float32))
    v_host = synth.round_bf16(g.standard_normal(shape, dtype=np.float32))
    paths = np.full((b, trj.PATH_STRIDE), -1, np.int32)
    for i, (p, k) in enumerate(zip(parents, ks)):
        rows = synth.random_path(seed + i, p, k)
        paths[i, :k + 1] = rows
    k_dev, v_dev = to_dev(k_host, dtype), to_dev(v_host, dtype)
    seq_len = i32(prefixes)
    trj.compact_rows(k_dev, v_dev, seq_len, i32(ks), i32(paths))
    torch.cuda.synchronize()
    for i in range(b):
        new_len = oracle.compact_rows(k_host[:, i], prefixes[i], paths[i, :ks[i] + 1])
        oracle.compact_rows(v_host[:, i], prefixes[i], paths[i, :ks[i] + 1])
        assert int(seq_len[i]) == new_len == prefixes[i] + ks[i] + 1
        # rows [0, new_len) are defined by the method; rows beyond are unspecified scratch
        np.testing.assert_array_equal(k_dev[:, i, :, :new_len].float().cpu().numpy(), k_host[:, i, :, :new_len])
        np.testing.assert_array_equal(v_dev[:, i, :, :new_len].float().cpu().numpy(), v_host[:, i, :, :new_len])


def test_compaction_config4(trj):
    parent = synth.random_tree(3, 128, 8, 4)
    for k in range(1, 9):
        check_compaction(trj, 30 + k, 1, 32, 128, "bf16", [8192], [parent], [k], 8192 + 128)


def test_compaction_ragged_multi_layer(trj):
    s, m = synth.ragged_batch(4, 8, (256, 4096), (16, 64))
    parents = [synth.random_tree(40 + i, int(mi), 6, 3) for i, mi in enumerate(m)]
    ks = [int(k) for k in synth.stream(4, "ks").integers(0, 7, size=8)]
    ks[0], ks[1] = 0, 6
    check_compaction(trj, 5, 3, 4, 128, "bf16", (s // 8).tolist(), parents, ks, 600)
    check_compaction(trj, 6, 2, 2, 64, "f32", (s // 16).tolist(), parents, ks, 400)


def test_compaction_long_chain_overlapping_ranges(trj):
    """k = 100 on a 128-row tree: source and destination row ranges overlap heavily."""
    parent = np.array([-1] + [max(0, i - 1 - (i % 5 == 0)) for i in range(1, 128)], np.int32)
    depth = synth.node_depths(parent)
    check_compaction(trj, 9, 2, 2, 128, "bf16", [37], [parent], [int(depth.max())], 37 + 128)


# ----------------------------------------------------------------------------- projection GEMM
@pytest.mark.parametrize("dtype,m,n,k", [
    ("bf16", 33, 512, 4096), ("bf16", 1, 130, 688), ("f32", 11, 1376, 256), ("bf16", 128, 257, 1104), ("f32", 70, 64, 688),
    # shapes the tcgen05 kernel takes: K >= 64, K % 8 == 0, N % 4 == 0; ragged N tiles, one k-block, deep split-K
    ("bf16", 48, 384, 64), ("bf16", 17, 132, 128), ("bf16", 33, 12288, 4096), ("bf16", 128, 4096, 11008),
    ("bf16", 1, 32000, 4096), ("bf16", 64, 22016, 4096), ("bf16", 16, 128, 8192), ("bf16", 100, 1000, 192),
    # more rows than one accumulator holds: row blocks (ragged last block, several K ranges, many blocks)
    ("bf16", 129, 512, 256), ("bf16", 257, 128, 64), ("bf16", 300, 260, 192), ("bf16", 512, 1024, 4096),
    ("bf16", 2048, 4096, 512), ("bf16", 1000, 384, 2048),
    # K that ends inside a 64-wide block (both operands read zeros past K): an eighth of the 7B feed-forward width
    ("bf16", 33, 4096, 1376), ("bf16", 7, 64, 72), ("bf16", 128, 512, 688), ("bf16", 300, 260, 200),
])
def test_gemm(trj, dtype, m, n, k):
    g = synth.stream(m * n, "gemm")
    x = g.standard_normal((m, k), dtype=np.float32)
    w = g.standard_normal((n, k), dtype=np.float32) * 0.02
    if dtype == "bf16":
        x, w = synth.round_bf16(x), synth.round_bf16(w)
    ws = torch.zeros(trj.lib().trj_gemm_workspace(m, n, k), dtype=torch.uint8, device="cuda")
    y = trj.gemm(to_dev(x, dtype), to_dev(w, dtype), workspace=ws).cpu().numpy()
    assert int(ws[:4].view(torch.int32)[0]) == 0           # no device-side wait expired
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.abs(y - ref).max() <= 1e-4 * max(1.0, np.abs(ref).max())
