"""The verification step with the decoder's weights split over ranks (heads and feed-forward columns), against the
CPU oracle of the WHOLE model.

All ranks' contexts live on the one GPU of the test and are stepped in lock-step; the sum over ranks that an
all-reduce would do between two segments is a plain sum of the ranks' exchange buffers.  Nothing runs
concurrently, so this checks the sharding and the segment boundaries, not a collective.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import anc_dev, i32

pytestmark = pytest.mark.gpu
MARGIN = 1e-2


def build(trj, cfg, seed, world, max_seq=256, max_rows=64):
    from paper_2406_17404_b200 import tp
    from paper_2406_17404_b200.decode import upload_weights
    layers = [synth.layer_weights(cfg, seed, l) for l in range(cfg.n_layers)]
    glob = synth.global_weights(cfg, seed)
    dl, dg = upload_weights(cfg, layers, glob)
    ranks = []
    for r in range(world):
        c, l, g = tp.shard_weights(cfg, dl, dg, r, world)
        ranks.append(trj.Model(c, l, g, max_batch=1, max_seq=max_seq, max_rows=max_rows))
    f64 = lambda d: {k: np.asarray(v, np.float64) for k, v in d.items()}
    return ranks, oracle.Decoder(cfg, [f64(l) for l in layers], f64(glob))


@pytest.mark.parametrize("cfg_name,world,tol", [("tiny", 2, 1e-3), ("tiny", 4, 1e-3), ("tiny_gqa", 2, 1e-3),
                                                ("7b", 2, 2e-2), ("7b", 4, 2e-2), ("llama3", 4, 2e-2)])
def test_sharded_step_equals_the_whole_model(trj, cfg_name, world, tol):
    from oracle.model import verify_step as oracle_step
    from paper_2406_17404_b200 import tp
    cfg = {"tiny": synth.TINY, "tiny_gqa": synth.TINY_GQA, "7b": synth.LLAMA7B.with_layers(2),
           "llama3": synth.LLAMA3_8B.with_layers(2)}[cfg_name]
    if cfg_name == "llama3":
        cfg = replace(cfg, vocab=32000)               # the LM head is not what is sharded
    ranks, dec = build(trj, cfg, 21, world)
    # prompt: 150 tokens = three chain chunks of at most 64 rows through the segment calls
    prompt = synth.prompt(31, 150, cfg.vocab)
    first = int(tp.prefill_local(ranks, torch.from_numpy(np.asarray(prompt, np.int32))).item())
    cache = dec.new_cache(256)
    lg = dec.forward_rows(cache, prompt, synth.chain_parents(len(prompt)))
    cache.seq_len = len(prompt)
    root = int(oracle.node_argmax(lg[-1:])[0])
    if oracle.top2_margin(lg[-1:])[0] >= MARGIN:
        assert first == root
    assert all(int(m.seq_len[0]) == len(prompt) for m in ranks)
    # every rank's cache holds its own K/V heads of the prompt
    hk = cfg.kv_heads // world
    lim = 1e-4 if cfg.dtype == "f32" else 0.07
    for r, m in enumerate(ranks):
        got = m.k_cache[:, 0, :, :len(prompt)].double().cpu().numpy()
        assert np.abs(got - cache.k[:, r * hk:(r + 1) * hk, :len(prompt)]).max() <= lim, r
    # one verification step over a random tree with planted drafts
    rows = 49
    parent = synth.random_tree(41, rows, 6, 3)
    tokens = synth.prompt(51, rows, cfg.vocab); tokens[0] = root
    probe = dec.new_cache(256); probe.k[:], probe.v[:], probe.seq_len = cache.k, cache.v, cache.seq_len
    pred0 = oracle.node_argmax(dec.forward_rows(probe, tokens, parent))
    g = synth.stream(21, "tp-plant")
    for i in range(1, rows):
        if g.random() < 0.5:
            tokens[i] = pred0[parent[i]]
    want = oracle_step(dec, cache, tokens, parent)
    depth, anc = trj.tree_from_parents(parent)
    d_tok, d_par, d_dep, d_off = i32(tokens), i32(parent), i32(depth), i32([0, rows])
    outs = tp.verify_step_local(ranks, d_tok, d_par, d_dep, anc_dev(anc), d_off, max_rows=rows,
                                max_len=len(prompt) + rows, want_logits=True, want_margin=True)
    torch.cuda.synchronize()
    for m in ranks:
        m.device_status()
    logits = outs[0]["logits"].cpu().numpy()
    assert np.abs(logits - want["logits"]).max() <= tol
    safe = oracle.top2_margin(want["logits"]) >= MARGIN
    pred = outs[0]["node_argmax"].cpu().numpy()
    np.testing.assert_array_equal(pred[safe], want["pred"][safe])
    for o in outs[1:]:                 # every rank holds the same residual stream, hence the same bits
        assert torch.equal(o["logits"], outs[0]["logits"]) and torch.equal(o["node_argmax"], outs[0]["node_argmax"])
    # acceptance and compaction, rank by rank on the rank's own cache slice
    for r, m in enumerate(ranks):
        acc = m.accept(d_tok, d_par, d_dep, d_off, outs[r]["node_argmax"])
        m.compact_kv(acc["k_acc"], acc["path"])
        k = int(acc["k_acc"][0]); path = acc["path"][0, :k + 1].tolist()
        assert (k, path, int(acc["bonus"][0])) == oracle.accept_path(tokens, parent, pred)
        if safe.all():
            assert (k, path) == (want["k"], want["path"])
            n = len(prompt) + k + 1
            assert int(m.seq_len[0]) == n == cache.seq_len
            got = m.v_cache[:, 0, :, :n].double().cpu().numpy()
            assert np.abs(got - cache.v[:, r * hk:(r + 1) * hk, :n]).max() <= lim
    for m in ranks:
        m.close()


def test_one_rank_is_the_plain_step(trj):
    """A single "rank" holding the whole model, walked segment by segment, against trj_verify_step itself: the
    segment boundaries change only the order of a few fp32 additions."""
    from paper_2406_17404_b200 import tp
    cfg = synth.LLAMA7B.with_layers(2)
    ranks, _ = build(trj, cfg, 22, 1)
    m = ranks[0]
    prompt = torch.from_numpy(np.asarray(synth.prompt(32, 90, cfg.vocab), np.int32))
    m.prefill(prompt.cuda())
    rows = 33
    parent = synth.random_tree(42, rows, 5, 2)
    tokens = synth.prompt(52, rows, cfg.vocab)
    depth, anc = trj.tree_from_parents(parent)
    args = (i32(tokens), i32(parent), i32(depth), anc_dev(anc), i32([0, rows]))
    a = m.verify_step(*args, max_rows=rows, max_len=90 + rows, want_logits=True, want_margin=True)
    b = tp.verify_step_local([m], *args, max_rows=rows, max_len=90 + rows, want_logits=True)[0]
    torch.cuda.synchronize()
    assert (a["logits"] - b["logits"]).abs().max().item() <= 2e-3
    safe = a["margin"] >= MARGIN
    assert torch.equal(a["node_argmax"][safe], b["node_argmax"][safe])
    m.close()


def test_segment_calls_out_of_order_are_refused(trj):
    cfg = synth.TINY
    ranks, _ = build(trj, cfg, 23, 2)
    m = ranks[0]
    with pytest.raises(trj.TrjError):
        m.tp_segment(0)                               # no step begun
    rows = 5
    parent = synth.chain_parents(rows)
    depth, anc = trj.tree_from_parents(parent)
    m.tp_begin(i32(synth.prompt(1, rows, cfg.vocab)), i32(parent), i32(depth), anc_dev(anc), i32([0, rows]),
               max_rows=rows, max_len=rows)
    assert m.tp_segments() == 2 * cfg.n_layers + 1
    with pytest.raises(trj.TrjError):
        m.tp_segment(1)                               # 0 comes first
    m.tp_segment(0)
    assert tuple(m.tp_exchange_tensor().shape) == (rows, cfg.d_model)
    with pytest.raises(trj.TrjError):
        m.tp_finish()                                 # segments left
    torch.cuda.synchronize()
    for r in ranks:
        r.close()
