"""Host side of the tensor-parallel step, on CPU: the weight slices add up to the whole projections, and the rank
driver calls the collective between the segments (two gloo processes around a stand-in for the context)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import synth
from paper_2406_17404_b200 import tp


def host_layer(cfg, seed, l):
    return {k: torch.from_numpy(np.asarray(v, np.float32)) for k, v in synth.layer_weights(cfg, seed, l).items()}


@pytest.mark.parametrize("cfg,world", [(synth.TINY, 2), (synth.TINY, 4), (synth.TINY_GQA, 2)])
def test_slices_add_up_to_the_whole_projections(cfg, world):
    layer = host_layer(cfg, 5, 0)
    g = torch.Generator().manual_seed(3)
    D, H, Hkv, f = cfg.head_dim, cfg.n_heads, cfg.kv_heads, cfg.d_ff
    x = torch.randn(7, cfg.d_model, generator=g)
    qkv = x @ layer["wqkv"].T
    attn_out = torch.randn(7, H * D, generator=g)            # stands for the attention result, head-major
    act = torch.randn(7, f, generator=g)
    gate_up = x @ layer["w_gate_up"].T
    o_sum, down_sum = torch.zeros(7, cfg.d_model), torch.zeros(7, cfg.d_model)
    hq, hk, fr = H // world, Hkv // world, f // world
    sc = tp.shard_cfg(cfg, world)
    assert (sc.n_heads, sc.kv_heads, sc.d_ff, sc.d_model, sc.vocab) == (hq, hk, fr, cfg.d_model, cfg.vocab)
    for r in range(world):
        s = tp.shard_layer(cfg, layer, r, world)
        assert s["wqkv"].shape == ((hq + 2 * hk) * D, cfg.d_model) and s["wo"].shape == (cfg.d_model, hq * D)
        assert s["w_gate_up"].shape == (2 * fr, cfg.d_model) and s["w_down"].shape == (cfg.d_model, fr)
        got = x @ s["wqkv"].T
        # the rank's query heads, then its key heads, then its value heads; a rank's query heads read its own K/V heads
        torch.testing.assert_close(got[:, :hq * D], qkv[:, r * hq * D:(r + 1) * hq * D])
        torch.testing.assert_close(got[:, hq * D:(hq + hk) * D], qkv[:, H * D + r * hk * D:H * D + (r + 1) * hk * D])
        torch.testing.assert_close(got[:, (hq + hk) * D:], qkv[:, (H + Hkv) * D + r * hk * D:(H + Hkv) * D + (r + 1) * hk * D])
        group = H // Hkv
        assert [(r * hq + h) // group for h in range(hq)] == [r * hk + h // (hq // hk) for h in range(hq)]
        gu = x @ s["w_gate_up"].T
        torch.testing.assert_close(gu[:, :fr], gate_up[:, r * fr:(r + 1) * fr])
        torch.testing.assert_close(gu[:, fr:], gate_up[:, f + r * fr:f + (r + 1) * fr])
        o_sum += attn_out[:, r * hq * D:(r + 1) * hq * D] @ s["wo"].T
        down_sum += act[:, r * fr:(r + 1) * fr] @ s["w_down"].T
    torch.testing.assert_close(o_sum, attn_out @ layer["wo"].T, rtol=1e-4, atol=1e-4)
    torch.testing.assert_close(down_sum, act @ layer["w_down"].T, rtol=1e-4, atol=1e-4)


def test_ranks_that_do_not_divide_the_heads_are_refused():
    with pytest.raises(ValueError):
        tp.shard_cfg(synth.TINY, 3)
    with pytest.raises(ValueError):
        tp.shard_cfg(synth.TINY_GQA, 4)          # two K/V heads


class FakeRankModel:
    """Stands for a rank's context: segment s leaves (rank + 1) * (s + 1) + what the previous exchange summed to."""

    def __init__(self, rank, n_segments):
        self.rank, self.n, self.buf, self.calls = rank, n_segments, torch.zeros(2, 3), []

    def tp_begin(self, *a, **k): self.calls.append("begin")
    def tp_segments(self): return self.n
    def tp_exchange_tensor(self): return self.buf

    def tp_segment(self, s, stream=None):
        self.calls.append(("seg", s, float(self.buf[0, 0])))
        if s + 1 < self.n:
            self.buf = self.buf + (self.rank + 1) * (s + 1)

    def tp_finish(self, **k):
        self.calls.append("finish")
        return {"last": float(self.buf[0, 0])}


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        m = FakeRankModel(rank, 5)
        res = tp.TPRank(m, tp.group_all_reduce()).verify_step(None, None, None, None, None, max_rows=1, max_len=1)
        out.put((rank, res["last"], m.calls))
    finally:
        dist.destroy_process_group()


def test_rank_driver_sums_between_segments_over_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs: p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60); assert p.exitcode == 0
    # after segment s both ranks hold world * previous + (1 + 2) * (s + 1): 3, 12, 33, 78
    want, seen = [], 0.0
    for s in range(4):
        seen = 2 * seen + 3 * (s + 1); want.append(seen)
    for rank, last, calls in got:
        assert last == want[-1]
        assert calls[0] == "begin" and calls[-1] == "finish"
        assert [c[1] for c in calls[1:-1]] == [0, 1, 2, 3, 4]
        assert [c[2] for c in calls[1:-1]] == [0.0] + want          # what each segment found in the buffer
