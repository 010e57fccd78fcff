"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

Each test names the passage it rests on.  None of them re-types an oracle
formula: they use invariants of the method (Eq. 1, Sections 2.1, 2.2, 3.3,
Appendix B), closed forms, brute force, hand-worked cases and an independent
library decoder.
"""
import itertools
import json
import os

import numpy as np
import pytest

import oracle
import synth
from oracle.model import rmsnorm, rope, silu, verify_step

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def tiny_decoder(seed=0, cfg=synth.TINY):
    layers = [synth.layer_weights(cfg, seed, l) for l in range(cfg.n_layers)]
    return oracle.Decoder(cfg, layers, synth.global_weights(cfg, seed))


@pytest.fixture(scope="module")
def dec():
    return tiny_decoder()


@pytest.fixture(scope="module")
def ar_tokens(dec):
    pr = synth.prompt(0, 64, dec.cfg.vocab)
    return pr, oracle.autoregressive_greedy(dec, pr, 48)


# ---------------------------------------------------------------- Section 2.2 / Appendix B
def test_chain_tree_is_causal_forward(dec):
    """A tree that is one chain is an ordinary sequence: logits equal the token-by-token forward."""
    toks = synth.prompt(3, 24, dec.cfg.vocab)
    c1 = dec.new_cache(32)
    chain = dec.forward_rows(c1, toks, synth.chain_parents(len(toks)))
    c2 = dec.new_cache(32)
    for i, t in enumerate(toks):
        row = dec.forward_rows(c2, [int(t)], [-1])
        c2.seq_len += 1
        np.testing.assert_allclose(chain[i], row[0], rtol=0, atol=1e-10)
    np.testing.assert_allclose(c1.k[:, :, :24], c2.k[:, :, :24], rtol=0, atol=1e-12)
    np.testing.assert_allclose(c1.v[:, :, :24], c2.v[:, :, :24], rtol=0, atol=1e-12)


def test_chain_attention_matches_library_causal_attention():
    """Chain tree over a prefix == causal scaled-dot-product attention of a library routine."""
    import torch
    t = synth.qkv(1, 3, 16, 10, 7, dtype="f32")
    out = oracle.tree_attention(t["q"], t["k_prefix"], t["v_prefix"], t["k_tree"], t["v_tree"],
                                synth.chain_parents(7))
    q = torch.tensor(t["q"], dtype=torch.float64).permute(1, 0, 2)[None]          # [1,H,M,D]
    k = torch.cat([torch.tensor(t["k_prefix"]), torch.tensor(t["k_tree"])], 1).double()[None]
    v = torch.cat([torch.tensor(t["v_prefix"]), torch.tensor(t["v_tree"])], 1).double()[None]
    allow = torch.ones(7, 17, dtype=torch.bool)
    allow[:, 10:] = torch.tril(torch.ones(7, 7, dtype=torch.bool))
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=allow)
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_subtree_independence_and_row_permutation(dec):
    """Rows outside a row's ancestor set do not influence it; relabelling rows changes nothing."""
    parent = synth.random_tree(5, 12, 4, 3)
    toks = synth.prompt(5, 12, dec.cfg.vocab)
    base_cache = dec.new_cache(40)
    dec.forward_rows(base_cache, synth.prompt(6, 9, dec.cfg.vocab), synth.chain_parents(9))
    base_cache.seq_len = 9

    def run(tokens, par):
        c = dec.new_cache(40)
        c.k[:], c.v[:], c.seq_len = base_cache.k, base_cache.v, 9
        return dec.forward_rows(c, tokens, par)

    full = run(toks, parent)
    mask = oracle.ancestor_mask(parent)
    for i in (3, 7, 11):
        keep = np.nonzero(mask[i])[0]                      # ancestors-or-self, ascending
        remap = {int(r): n for n, r in enumerate(keep)}
        sub_parent = [-1] + [remap[int(parent[r])] for r in keep[1:]]
        sub = run(toks[keep], sub_parent)
        np.testing.assert_allclose(sub[-1], full[i], rtol=0, atol=1e-10)
    # a different topological order of the same tree
    order = [0] + sorted(range(1, 12), key=lambda r: (synth.node_depths(parent)[r], -r))
    inv = {r: n for n, r in enumerate(order)}
    p2 = [-1] + [inv[int(parent[r])] for r in order[1:]]
    perm = run(toks[order], p2)
    np.testing.assert_allclose(perm, full[order], rtol=0, atol=1e-10)


def test_attention_closed_forms():
    """One visible key -> its value; equal keys -> the mean of the visible values; empty prefix works."""
    g = np.random.default_rng(0)
    h, d = 2, 8
    q = g.standard_normal((1, h, d))
    kt, vt = g.standard_normal((h, 1, d)), g.standard_normal((h, 1, d))
    empty = np.zeros((h, 0, d))
    out = oracle.tree_attention(q, empty, empty, kt, vt, [-1])
    np.testing.assert_allclose(out[0], vt[:, 0], atol=1e-14)
    # all keys equal: weights are uniform over the visible set
    parent = [-1, 0, 0, 1]
    q = g.standard_normal((4, h, d))
    kp = np.tile(g.standard_normal((h, 1, d)), (1, 5, 1))
    vp = g.standard_normal((h, 5, d))
    ktr = np.tile(kp[:, :1], (1, 4, 1))
    vtr = g.standard_normal((h, 4, d))
    out = oracle.tree_attention(q, kp, vp, ktr, vtr, parent)
    vis3 = [0, 1, 3]
    want = (vp.sum(1) + vtr[:, vis3].sum(1)) / (5 + 3)
    np.testing.assert_allclose(out[3], want, atol=1e-13)
    want2 = (vp.sum(1) + vtr[:, [0, 2]].sum(1)) / (5 + 2)
    np.testing.assert_allclose(out[2], want2, atol=1e-13)


def test_attention_is_shift_and_scale_consistent():
    """softmax is invariant to adding a constant key component along q; huge score -> one-hot."""
    g = np.random.default_rng(1)
    h, d = 1, 4
    q = np.zeros((1, h, d)); q[0, 0, 0] = 50.0
    kp = np.zeros((h, 3, d)); kp[0, 1, 0] = 10.0          # score 250 vs 0: row 1 dominates
    vp = g.standard_normal((h, 3, d))
    kt, vt = np.zeros((h, 1, d)), g.standard_normal((h, 1, d))
    out = oracle.tree_attention(q, kp, vp, kt, vt, [-1])
    np.testing.assert_allclose(out[0, 0], vp[0, 1], atol=1e-12)


# ---------------------------------------------------------------- model-side conventions
def test_rope_invariants():
    """Rotation preserves norms, is the identity at position 0, and q.k depends on pos difference only."""
    g = np.random.default_rng(2)
    x, y = g.standard_normal((1, 2, 16)), g.standard_normal((1, 2, 16))
    np.testing.assert_allclose(rope(x, np.array([0]), 1e4), x, atol=1e-15)
    for p in (1, 17, 400):
        np.testing.assert_allclose(np.linalg.norm(rope(x, np.array([p]), 1e4), axis=-1),
                                   np.linalg.norm(x, axis=-1), atol=1e-12)
    dots = [np.sum(rope(x, np.array([p + 5]), 1e4) * rope(y, np.array([p]), 1e4), -1) for p in (0, 3, 111)]
    np.testing.assert_allclose(dots[0], dots[1], atol=1e-11)
    np.testing.assert_allclose(dots[0], dots[2], atol=1e-11)
    # lowest pair rotates by exactly pos radians (frequency theta^0 = 1), pairing (0, D/2)
    e = np.zeros((1, 1, 16)); e[0, 0, 0] = 1.0
    r = rope(e, np.array([2]), 1e4)[0, 0]
    np.testing.assert_allclose([r[0], r[8]], [np.cos(2.0), np.sin(2.0)], atol=1e-15)
    # highest pair rotates by pos * theta^(-(D-2)/D)
    e = np.zeros((1, 1, 16)); e[0, 0, 7] = 1.0
    r = rope(e, np.array([3]), 1e4)[0, 0]
    ang = 3 * 1e4 ** (-14 / 16)
    np.testing.assert_allclose([r[7], r[15]], [np.cos(ang), np.sin(ang)], atol=1e-15)


def test_rmsnorm_and_silu_closed_forms():
    x = np.array([[3.0, -4.0, 0.0, 0.0]])
    np.testing.assert_allclose(rmsnorm(x, np.ones(4), 0.0), x / 2.5, atol=1e-15)      # rms = sqrt(25/4)
    np.testing.assert_allclose(rmsnorm(7 * x, 2 * np.ones(4), 0.0), 2 * x / 2.5, atol=1e-15)
    assert abs(rmsnorm(np.array([[1e-3]]), np.ones(1), 1e-5)[0, 0] - 1e-3 / np.sqrt(1e-6 + 1e-5)) < 1e-15
    assert silu(np.array([0.0]))[0] == 0.0
    np.testing.assert_allclose(silu(np.array([40.0, -40.0])), [40.0, 0.0], atol=1e-15)
    np.testing.assert_allclose(silu(np.array([1.0])), 1.0 / (1.0 + np.exp(-1.0)), atol=1e-16)


def test_matches_independent_library_decoder(dec):
    """Causal logits of the tiny config equal those of transformers' LLaMA implementation in fp64."""
    torch = pytest.importorskip("torch")
    tf = pytest.importorskip("transformers")
    cfg = dec.cfg
    hc = tf.LlamaConfig(vocab_size=cfg.vocab, hidden_size=cfg.d_model, intermediate_size=cfg.d_ff,
                        num_hidden_layers=cfg.n_layers, num_attention_heads=cfg.n_heads,
                        num_key_value_heads=cfg.n_heads, head_dim=cfg.head_dim, rms_norm_eps=cfg.rms_eps,
                        rope_theta=cfg.rope_theta, attention_bias=False, mlp_bias=False,
                        tie_word_embeddings=False, max_position_embeddings=256)
    hf = tf.LlamaForCausalLM(hc).double().eval()
    hd = cfg.n_heads * cfg.head_dim
    sd = {"model.embed_tokens.weight": dec.glob["embed"], "lm_head.weight": dec.glob["lm_head"],
          "model.norm.weight": dec.glob["final_norm"]}
    for l in range(cfg.n_layers):
        w, p = dec.layers[l], f"model.layers.{l}."
        sd[p + "self_attn.q_proj.weight"] = w["wqkv"][:hd]
        sd[p + "self_attn.k_proj.weight"] = w["wqkv"][hd:2 * hd]
        sd[p + "self_attn.v_proj.weight"] = w["wqkv"][2 * hd:]
        sd[p + "self_attn.o_proj.weight"] = w["wo"]
        sd[p + "mlp.gate_proj.weight"] = w["w_gate_up"][:cfg.d_ff]
        sd[p + "mlp.up_proj.weight"] = w["w_gate_up"][cfg.d_ff:]
        sd[p + "mlp.down_proj.weight"] = w["w_down"]
        sd[p + "input_layernorm.weight"] = w["attn_norm"]
        sd[p + "post_attention_layernorm.weight"] = w["mlp_norm"]
    missing = hf.load_state_dict({k: torch.tensor(np.asarray(v), dtype=torch.float64) for k, v in sd.items()},
                                 strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k and "inv_freq" not in k]
    toks = synth.prompt(9, 20, cfg.vocab)
    with torch.no_grad():
        ref = hf(torch.tensor(toks[None].astype(np.int64))).logits[0].numpy()
    got = dec.forward_rows(dec.new_cache(32), toks, synth.chain_parents(20))
    # the library builds its rotary table in fp32 whatever the model dtype, hence 1e-6 and not 1e-12;
    # a wrong pairing, base, eps or mask moves the logits by ~1e-1
    np.testing.assert_allclose(got, ref, rtol=0, atol=2e-6)


def _load_into_library_decoder(tf, torch, dec):
    cfg = dec.cfg
    hc = tf.LlamaConfig(vocab_size=cfg.vocab, hidden_size=cfg.d_model, intermediate_size=cfg.d_ff,
                        num_hidden_layers=cfg.n_layers, num_attention_heads=cfg.n_heads,
                        num_key_value_heads=cfg.kv_heads, head_dim=cfg.head_dim, rms_norm_eps=cfg.rms_eps,
                        rope_theta=cfg.rope_theta, attention_bias=False, mlp_bias=False,
                        tie_word_embeddings=False, max_position_embeddings=256)
    hf = tf.LlamaForCausalLM(hc).double().eval()
    hd, kvd = cfg.n_heads * cfg.head_dim, cfg.kv_heads * cfg.head_dim
    sd = {"model.embed_tokens.weight": dec.glob["embed"], "lm_head.weight": dec.glob["lm_head"],
          "model.norm.weight": dec.glob["final_norm"]}
    for l in range(cfg.n_layers):
        w, p = dec.layers[l], f"model.layers.{l}."
        sd[p + "self_attn.q_proj.weight"] = w["wqkv"][:hd]
        sd[p + "self_attn.k_proj.weight"] = w["wqkv"][hd:hd + kvd]
        sd[p + "self_attn.v_proj.weight"] = w["wqkv"][hd + kvd:]
        sd[p + "self_attn.o_proj.weight"] = w["wo"]
        sd[p + "mlp.gate_proj.weight"] = w["w_gate_up"][:cfg.d_ff]
        sd[p + "mlp.up_proj.weight"] = w["w_gate_up"][cfg.d_ff:]
        sd[p + "mlp.down_proj.weight"] = w["w_down"]
        sd[p + "input_layernorm.weight"] = w["attn_norm"]
        sd[p + "post_attention_layernorm.weight"] = w["mlp_norm"]
    missing = hf.load_state_dict({k: torch.tensor(np.asarray(v), dtype=torch.float64) for k, v in sd.items()},
                                 strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k and "inv_freq" not in k]
    return hf


def test_grouped_query_attention_matches_library_decoder():
    """Grouped-query attention (the LLaMA-3 family of Table 2): 4 query heads over 2 K/V heads on the tiny shape
    give the causal logits of transformers' LLaMA with num_key_value_heads = 2."""
    torch = pytest.importorskip("torch")
    tf = pytest.importorskip("transformers")
    dec = tiny_decoder(3, synth.TINY_GQA)
    hf = _load_into_library_decoder(tf, torch, dec)
    toks = synth.prompt(19, 20, dec.cfg.vocab)
    with torch.no_grad():
        ref = hf(torch.tensor(toks[None].astype(np.int64))).logits[0].numpy()
    got = dec.forward_rows(dec.new_cache(32), toks, synth.chain_parents(20))
    np.testing.assert_allclose(got, ref, rtol=0, atol=2e-6)


def test_grouped_query_attention_is_multi_head_attention_with_repeated_kv():
    """A grouped-query model is the multi-head model whose K/V projection rows are repeated once per query head of
    the group: same logits and, head for head, the same cache rows, on a branching tree over a non-empty cache."""
    from dataclasses import replace
    cfg = synth.TINY_GQA
    dec = tiny_decoder(5, cfg)
    h, kv, d = cfg.n_heads, cfg.kv_heads, cfg.head_dim
    rep = np.repeat(np.arange(kv), h // kv)                  # K/V head of every query head
    wide_layers = []
    for w in dec.layers:
        wq, wk, wv = w["wqkv"][:h * d], w["wqkv"][h * d:(h + kv) * d], w["wqkv"][(h + kv) * d:]
        wk = wk.reshape(kv, d, -1)[rep].reshape(h * d, -1)
        wv = wv.reshape(kv, d, -1)[rep].reshape(h * d, -1)
        wide_layers.append({**w, "wqkv": np.concatenate([wq, wk, wv], 0)})
    wide = oracle.Decoder(replace(cfg, n_kv_heads=0), wide_layers, dec.glob)
    prompt = synth.prompt(6, 12, cfg.vocab)
    parent = synth.random_tree(6, 14, 4, 3)
    tokens = synth.prompt(7, 14, cfg.vocab)
    outs = []
    for model in (dec, wide):
        cache = model.new_cache(40)
        model.forward_rows(cache, prompt, synth.chain_parents(12))
        cache.seq_len = 12
        outs.append((model.forward_rows(cache, tokens, parent), cache))
    np.testing.assert_allclose(outs[0][0], outs[1][0], rtol=0, atol=1e-12)
    np.testing.assert_allclose(outs[0][1].k[:, rep], outs[1][1].k, rtol=0, atol=1e-13)
    assert outs[0][1].k.shape[1] == kv and outs[1][1].k.shape[1] == h


def test_grouped_query_tr_jacobi_equals_autoregressive():
    """Eq. 1 with grouped-query attention: greedy TR-Jacobi commits the autoregressive tokens."""
    dec = tiny_decoder(3, synth.TINY_GQA)
    pr = synth.prompt(2, 40, dec.cfg.vocab)
    ar = oracle.autoregressive_greedy(dec, pr, 24)
    got = oracle.tr_jacobi_generate(dec, pr, 24, 4, 2, 3, lambda s, n: synth.noise_draws(8, s, n))
    assert got == ar


# ---------------------------------------------------------------- Appendix B: top-K siblings
def test_node_topk_order_ties_and_reduction_to_argmax():
    logits = np.array([[0.5, 2.0, 2.0, -1.0, 2.0, 0.5],      # three-way tie at the top, two-way tie below it
                       [3.0, 1.0, 0.0, 7.0, 7.0, -2.0],
                       [1.0, 1.0, 1.0, 1.0, 1.0, 1.0]])
    np.testing.assert_array_equal(oracle.node_topk(logits, 4), [[1, 2, 4, 0], [3, 4, 0, 1], [0, 1, 2, 3]])
    g = synth.stream(4, "topk")
    x = g.standard_normal((7, 500))
    top = oracle.node_topk(x, 10)
    np.testing.assert_array_equal(top[:, 0], oracle.node_argmax(x))          # K = 1 is the greedy prediction
    np.testing.assert_array_equal(oracle.node_topk(x, 1)[:, 0], oracle.node_argmax(x))
    torch = pytest.importorskip("torch")                      # distinct values: the library's top-k gives the same ids
    np.testing.assert_array_equal(top, torch.topk(torch.from_numpy(x), 10, dim=1).indices.numpy())


def test_refill_tree_hand_worked_and_chain_reduces_to_window_refill():
    # template: root; rows 1, 2 = rank 0, 1 under the root; row 3 = retrieval slot 0; rows 4, 5 = rank 0, 1 under row 1;
    # row 6 = rank 0 under row 4
    parent = [-1, 0, 0, 0, 1, 1, 4]
    rank = [0, 0, 1, -1, 0, 1, 0]
    topk = np.arange(7 * 3).reshape(7, 3) + 100               # row i offers 100 + 3i, 101 + 3i, 102 + 3i
    ctx = [9, 8, 7, 6]
    draws = [5, 2, 3, 0, 1, 7]
    # winner = root: the rows below it are 1, 4, 6 -> depth 1 from row 1, depth 2 from row 4, depth 3 from row 6
    assert oracle.continuation_rows(parent, 0) == [1, 4, 6]
    assert oracle.refill_tree(parent, rank, topk, 0, ctx, draws, [55]) == [103, 104, 55, 112, 113, 118]
    # winner = row 1: below it 4, 6 -> depth 1 from row 4, depth 2 from row 6, depth 3 is noise (row 6 uses draws[5])
    assert oracle.refill_tree(parent, rank, topk, 1, ctx, draws, [55]) == [112, 113, 55, 118, 119, ctx[7 % 4]]
    # winner = row 2 (a leaf): everything but the retrieval slot is noise
    assert oracle.refill_tree(parent, rank, topk, 2, ctx, draws, [55]) == [ctx[5 % 4], ctx[2], 55, ctx[0], ctx[1], ctx[3]]
    # a chain with ranks 0 is the Jacobi window
    g = synth.stream(6, "chain")
    for best in range(6):
        pred = g.integers(0, 1000, size=6)
        d = g.integers(0, 1000, size=5)
        chain = synth.chain_parents(6)
        want = oracle.refill_window(chain, pred, best, 5, ctx, d[:5])
        got = oracle.refill_tree(chain, [0] * 6, pred[:, None], best, ctx, np.concatenate([np.zeros(best, np.int64), d]), [])
        # refill_window numbers its noise draws from the first unfilled slot of the window, refill_tree by row
        filled = 5 - best
        assert got[:filled] == want[:filled]


@pytest.mark.parametrize("seed,n_nodes,top_k,n_retr", [(0, 63, 10, 5), (1, 20, 5, 0), (2, 12, 6, 3)])
def test_top_k_tree_decoding_equals_autoregressive(dec, ar_tokens, seed, n_nodes, top_k, n_retr):
    """Eq. 1 on a static template with top-K siblings and a retrieval path (Appendix B): same tokens as greedy
    autoregressive decoding, whatever the template, K or the noise."""
    prompt, ar = ar_tokens
    parent, rank = synth.tree_template(seed, n_nodes, 4, 10, n_retr)
    assert len(parent) == 1 + n_nodes + n_retr and rank.max() < top_k
    trace = []
    got = oracle.tr_jacobi_generate_tree(dec, prompt, 40, parent, rank, top_k, n_retr,
                                         lambda s, n: synth.noise_draws(seed, s, n), trace=trace)
    assert got == ar[:40]
    assert len(trace) <= 40
    # siblings of one parent hold distinct candidates whenever they come from a prediction (same source row, different rank)
    for rec in trace[1:]:
        tok, par = rec["tokens"], rec["parent"]
        assert len(tok) == len(parent)


# ---------------------------------------------------------------- Eq. 1, Sections 2.1 and 3.3
@pytest.mark.parametrize("width,n_br,br_len,seed", [(4, 2, 3, 0), (5, 3, 3, 1), (3, 0, 0, 2), (1, 1, 5, 3), (8, 1, 2, 4)])
def test_tr_jacobi_equals_autoregressive(dec, ar_tokens, width, n_br, br_len, seed):
    """Greedy TR-Jacobi commits exactly the autoregressive greedy tokens, for any window/retrieval/noise."""
    pr, ar = ar_tokens
    trace = []
    out = oracle.tr_jacobi_generate(dec, pr, 48, width, n_br, br_len,
                                    lambda s, n: synth.noise_draws(seed, s, n), trace=trace)
    assert out == ar
    # at least one token per step (an autoregressive step has #MAT 1.00, Table 2)
    assert all(r["k"] >= 0 and len(r["path"]) == r["k"] + 1 for r in trace)
    assert len(trace) <= 48
    assert all(len(r["tokens"]) == 1 + width + n_br * br_len for r in trace)


def test_random_trees_commit_autoregressive_tokens_and_cache(dec, ar_tokens):
    """Arbitrary tree shapes with partly-correct drafts: committed tokens == AR, compacted cache == AR cache."""
    pr, ar = ar_tokens
    truth = [int(t) for t in pr] + ar
    cache = dec.new_cache(200)
    dec.forward_rows(cache, pr[:-1], synth.chain_parents(len(pr) - 1))
    cache.seq_len = len(pr) - 1
    committed = [int(t) for t in pr]                      # root = last prompt token, not cached yet
    step = 0
    ks = []
    while len(committed) < len(pr) + 30:
        step += 1
        parent = synth.random_tree(100 + step, 10, 4, 3, name="t")
        depth = synth.node_depths(parent)
        g = synth.stream(7, f"draft{step}")
        tokens = np.zeros(10, np.int32)
        tokens[0] = committed[-1]
        for i in range(1, 10):                            # true continuation with prob 0.7, else random
            true_tok = truth[len(committed) - 1 + depth[i]]
            tokens[i] = true_tok if g.random() < 0.7 else g.integers(0, dec.cfg.vocab)
        rec = verify_step(dec, cache, tokens, parent)
        committed += [int(tokens[r]) for r in rec["path"][1:]] + [rec["bonus"]]
        ks.append(rec["k"])
        assert committed == truth[:len(committed)]
        assert cache.seq_len == len(committed) - 1
    assert max(ks) >= 2 and min(ks) == 0 or len(set(ks)) > 1
    ref = dec.new_cache(200)
    n = cache.seq_len
    dec.forward_rows(ref, truth[:n], synth.chain_parents(n))
    np.testing.assert_allclose(cache.k[:, :, :n], ref.k[:, :, :n], rtol=0, atol=1e-10)
    np.testing.assert_allclose(cache.v[:, :, :n], ref.v[:, :, :n], rtol=0, atol=1e-10)


def test_true_drafts_are_fully_accepted(dec, ar_tokens):
    """If every draft is the true continuation, the whole depth is accepted (k = depth of the tree)."""
    pr, ar = ar_tokens
    truth = [int(t) for t in pr] + ar
    cache = dec.new_cache(120)
    dec.forward_rows(cache, pr[:-1], synth.chain_parents(len(pr) - 1))
    cache.seq_len = len(pr) - 1
    parent = synth.random_tree(11, 9, 4, 2)
    depth = synth.node_depths(parent)
    tokens = np.array([truth[len(pr) - 1 + d] for d in depth], np.int32)
    rec = verify_step(dec, cache, tokens, parent)
    assert rec["k"] == depth.max() == 4
    assert rec["bonus"] == truth[len(pr) + 4]


def test_jacobi_window_converges_within_width(dec, ar_tokens):
    """Section 2.1: a length-m window reaches its fixed point in at most m iterations.

    Iterating the same window positions (no commit), iteration t makes at least
    the first t window tokens equal the greedy continuation.
    """
    pr, ar = ar_tokens
    width = 5
    cache = dec.new_cache(100)
    dec.forward_rows(cache, pr, synth.chain_parents(len(pr)))
    cache.seq_len = len(pr)
    root = ar[0]
    window = [int(pr[i]) for i in range(width)]           # arbitrary initial guess
    for it in range(1, width + 1):
        tokens, parent = oracle.build_tree(root, window, [])
        pred = oracle.node_argmax(dec.forward_rows(cache, tokens, parent))
        window = [int(pred[i]) for i in range(width)]     # Jacobi update: y_i <- argmax P(. | y_<i)
        assert window[:it] == ar[1:1 + it]
    assert window == ar[1:1 + width]


def brute_force_accept(dec, cache_len, prompt_cache_tokens, tokens, parent):
    """Score every root-to-node path by plain sequential greedy decoding; keep the longest match."""
    depth = synth.node_depths(parent)
    best_len, best_tokens = 0, []
    need = int(depth.max()) + 1
    truth = oracle.autoregressive_greedy(dec, list(prompt_cache_tokens) + [int(tokens[0])], need)
    for node in range(len(parent)):
        path, j = [], node
        while j > 0:
            path.append(int(tokens[j])); j = int(parent[j])
        path.reverse()
        if path == truth[:len(path)] and len(path) > best_len:
            best_len, best_tokens = len(path), path
    return best_len, best_tokens, truth[best_len]


@pytest.mark.parametrize("seed", range(6))
def test_bruteforce_path_enumeration(dec, seed):
    """Tiny trees: enumerating all paths against sequential greedy decoding gives the same k, tokens, bonus."""
    ctx = synth.prompt(20 + seed, 12, dec.cfg.vocab)
    truth = oracle.autoregressive_greedy(dec, ctx, 6)
    m = 5 + seed
    parent = synth.random_tree(seed, m, 3, 3, name="bf")
    depth = synth.node_depths(parent)
    g = synth.stream(seed, "bf_tok")
    tokens = np.zeros(m, np.int32)
    tokens[0] = truth[0]
    for i in range(1, m):
        tokens[i] = truth[depth[i]] if g.random() < 0.6 else g.integers(0, dec.cfg.vocab)
    cache = dec.new_cache(40)
    dec.forward_rows(cache, ctx, synth.chain_parents(len(ctx)))
    cache.seq_len = len(ctx)
    rec = verify_step(dec, cache, tokens, parent)
    k, toks, bonus = brute_force_accept(dec, len(ctx), ctx, tokens, parent)
    assert rec["k"] == k
    assert [int(tokens[r]) for r in rec["path"][1:]] == toks
    assert rec["bonus"] == bonus


# ---------------------------------------------------------------- integer pieces, hand-worked
def test_accept_hand_worked_cases():
    with open(os.path.join(GOLDEN, "accept_cases.json")) as f:
        cases = json.load(f)["cases"]
    for c in cases:
        k, path, bonus = oracle.accept_path(c["tokens"], c["parent"], c["pred"])
        assert (k, path, bonus) == (c["k"], c["path"], c["bonus"]), c["name"]


def test_argmax_ties_and_margin():
    x = np.array([[0.0, 3.0, 3.0, 1.0], [5.0, 5.0, 5.0, 5.0], [-1.0, -2.0, -0.5, -0.75]])
    assert list(oracle.node_argmax(x)) == [1, 0, 2]
    np.testing.assert_allclose(oracle.top2_margin(x), [0.0, 0.0, 0.25])


def test_build_tree_layout_and_mask_bits():
    """Row 0 root, window as a chain, each retrieved branch as its own chain off the root (Section 3.3)."""
    tokens, parent = oracle.build_tree(9, [1, 2, 3], [[4, 5], [6, 7]])
    assert list(tokens) == [9, 1, 2, 3, 4, 5, 6, 7]
    assert list(parent) == [-1, 0, 1, 2, 0, 4, 0, 6]
    assert list(oracle.depths(parent)) == [0, 1, 2, 3, 1, 2, 1, 2]
    mask = oracle.ancestor_mask(parent)
    assert [list(np.nonzero(r)[0]) for r in mask] == [[0], [0, 1], [0, 1, 2], [0, 1, 2, 3], [0, 4], [0, 4, 5],
                                                      [0, 6], [0, 6, 7]]
    bits = oracle.pack_mask(mask)
    assert bits.shape == (8, 1)
    assert [int(b) for b in bits[:, 0]] == [0b1, 0b11, 0b111, 0b1111, 0b10001, 0b110001, 0b1000001, 0b11000001]
    # 70 rows: bit j lives in word j // 64
    chain = oracle.pack_mask(oracle.ancestor_mask(synth.chain_parents(70)))
    assert chain.shape == (70, 2) and int(chain[69, 0]) == 2 ** 64 - 1 and int(chain[69, 1]) == 0b111111
    with pytest.raises(ValueError):
        oracle.validate_tree([-1, 1])
    with pytest.raises(ValueError):
        oracle.validate_tree([0, 0])


def test_retrieve_hand_worked():
    """Prompt lookup: continuation of the most recent earlier occurrences of the tail (Section 3.3)."""
    ctx = [1, 2, 3, 4, 1, 2, 5, 6, 1, 2]
    draws = list(range(100, 112))
    # key (1,2): earlier occurrences at 4 (-> 5,6,1) and 0 (-> 3,4,1); most recent first
    assert oracle.retrieve(ctx, 2, 3, draws) == [[5, 6, 1], [3, 4, 1]]
    # three branches: two bigram matches, then the unigram key (2) adds nothing new -> ahead noise
    got = oracle.retrieve(ctx, 3, 2, draws)
    assert got[:2] == [[5, 6], [3, 4]]
    assert got[2] == [ctx[104 % 10], ctx[105 % 10]]
    # unigram fallback and a continuation that runs off the end
    ctx2 = [7, 8, 9, 7]
    assert oracle.retrieve(ctx2, 1, 4, [0, 1, 2, 3]) == [[8, 9, 7, ctx2[3 % 4]]]
    # no match at all: every slot is ahead noise over the context (Eq. 4)
    ctx3 = [1, 2, 3]
    assert oracle.retrieve(ctx3, 1, 2, [4, 5]) == [[ctx3[4 % 3], ctx3[5 % 3]]]


def test_refill_follows_the_winning_branch():
    """Next window = predictions below the winner on its branch, then ahead noise (Section 3.3)."""
    _, parent = oracle.build_tree(0, [0, 0, 0], [[0, 0]])              # rows: 0 | 1 2 3 | 4 5
    pred = [10, 11, 12, 13, 14, 15]
    ctx = [40, 41, 42]
    assert oracle.refill_window(parent, pred, 1, 3, ctx, [0, 1, 2]) == [12, 13, ctx[2]]
    assert oracle.refill_window(parent, pred, 4, 3, ctx, [0, 1, 2]) == [15, ctx[1], ctx[2]]
    assert oracle.refill_window(parent, pred, 0, 3, ctx, [0, 1, 2]) == [11, 12, 13]
    assert oracle.refill_window(parent, pred, 3, 3, ctx, [5, 6, 7]) == [ctx[2], ctx[0], ctx[1]]


def test_compact_rows_moves_path_rows():
    cache = np.arange(2 * 12 * 3, dtype=np.float64).reshape(2, 12, 3)
    before = cache.copy()
    new_len = oracle.compact_rows(cache, 4, [0, 2, 5])
    assert new_len == 7
    np.testing.assert_array_equal(cache[:, :4], before[:, :4])
    np.testing.assert_array_equal(cache[:, 4], before[:, 4])
    np.testing.assert_array_equal(cache[:, 5], before[:, 6])
    np.testing.assert_array_equal(cache[:, 6], before[:, 9])


def test_generators_are_reproducible_and_bf16_exact():
    a = synth.logits(3, 4, 64)
    b = synth.logits(3, 4, 64)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(synth.round_bf16(a), a)
    bits = synth.bf16_bits(a)
    back = (bits.astype(np.uint32) << 16).view(np.float32)
    np.testing.assert_array_equal(back, a)
    # ties-to-even on a value exactly between two bf16 numbers
    x = np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8], np.float32)
    np.testing.assert_array_equal(synth.round_bf16(x), np.array([1.0, 1.0 + 2 ** -6], np.float32))


# ---------------------------------------------------------------- bf16 storage of the attention operands
def test_store_bf16_matches_library_conversion_and_ties_to_even():
    import torch
    from oracle.model import store_bf16
    g = np.random.default_rng(0)
    x = g.standard_normal(50000) * np.exp(g.uniform(-20, 20, 50000))
    ref = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).double().numpy()
    np.testing.assert_array_equal(store_bf16(x), ref)
    np.testing.assert_array_equal(store_bf16(np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -1.0 - 2 ** -8])),
                                  [1.0, 1.0 + 2 ** -6, -1.0])


def test_bf16_model_rounds_only_the_attention_operands():
    """In a bf16 config the cache rows and q are bf16 values; TR-Jacobi still equals greedy AR decoding."""
    import dataclasses
    cfg = dataclasses.replace(synth.TINY, dtype="bf16")
    dec = tiny_decoder(3, cfg)
    pr = synth.prompt(3, 40, cfg.vocab)
    cache = dec.new_cache(64)
    dec.forward_rows(cache, pr, synth.chain_parents(40))
    np.testing.assert_array_equal(synth.round_bf16(cache.k[:, :, :40].astype(np.float32)), cache.k[:, :, :40])
    np.testing.assert_array_equal(synth.round_bf16(cache.v[:, :, :40].astype(np.float32)), cache.v[:, :, :40])
    ar = oracle.autoregressive_greedy(dec, pr, 30)
    out = oracle.tr_jacobi_generate(dec, pr, 30, 4, 2, 3, lambda s, n: synth.noise_draws(5, s, n))
    assert out == ar
