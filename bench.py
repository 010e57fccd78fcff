#!/usr/bin/env python
"""Benchmark of the TR-Jacobi verification step (one B200 per rank, replicas only).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload (N = 1 and every rank of N > 1): a LLaMA-2-7B-shaped random-init bf16 decoder, a 512-token
random prompt already prefilled, TR-Jacobi trees of 32 draft tokens + root (Jacobi window 5 plus nine
retrieved branches of 3).  One step = the whole hot path: tree build, verification forward over the 33
rows, per-node arg-max, longest-path acceptance, KV compaction.  Prints ONE JSON line.

`value`   draft tokens verified per second with the tree already resident in HBM (CUDA events).
`e2e`     the same metric through trj_step_host: host integers in, host result out, H2D/D2H inside.
`roofline` the projection kernels (they stream the 13.2 GB of weights): algorithmic bytes / device time.
`tree_attention` the op-level tree attention of the 64-row / prefix-1024 and 128-row / prefix-8192 cases.
`cpu_baseline` the CPU oracle timed on one full verification step (our arm) or, per timed step of the reference
           arm, on a bounded sample (two of the 32 layers + LM head) with the extrapolation stated separately.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WIDTH, N_BRANCHES, BRANCH_LEN = 5, 9, 3
TREE_ROWS = 1 + WIDTH + N_BRANCHES * BRANCH_LEN          # 33
DRAFTS = TREE_ROWS - 1                                   # 32 draft tokens per step
PROMPT = 512
METRIC = "draft_tokens_verified_per_s"
UNIT = "tokens/s"
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of ALL 129 projection launches of one step, from an ncu
# capture of the current projection kernel on a 4-layer model, scaled to 32 layers + the LM head: per layer 443.3 MB
# (QKV 102.4, output 65.1 incl. 30 MB of gate/up weights that it prefetches and that ncu's serialised timing counts
# again in the gate/up launch, gate/up 183.2, down 92.6), LM head 263.1 MB.  Set to None whenever that kernel changes.
GEMM_TRAFFIC_BYTES_PER_STEP = int(32 * 443.3e6 + 263.1e6)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.file = index, None, None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# --------------------------------------------------------------------------------------- our arm
def gemm_bytes_per_step(cfg, rows):
    """Algorithmic bytes of all projections of one verification step: every weight once (bf16), the
    split-bf16 activations in and the fp32 results out."""
    d, f, hd, v = cfg.d_model, cfg.d_ff, cfg.n_heads * cfg.head_dim, cfg.vocab
    per_layer = [(3 * hd, d, 2), (d, hd, 2), (2 * f, d, 2), (d, f, 2)]      # (N, K, activation halves)
    total = 0
    for n, k, halves in per_layer:
        total += cfg.n_layers * (n * k * 2 + rows * k * 2 * halves + rows * n * 4)
    total += v * d * 2 + rows * d * 2 * 2 + rows * v * 4
    return total


def graph_us(torch, fn, steps, warmup):
    """Average device time of one call of ``fn`` (a fixed launch sequence), replayed from a CUDA graph."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())        # what fn reads may still be in flight on the caller's stream
    with torch.cuda.stream(side):
        fn()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        fn()
    for _ in range(warmup):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / steps


def oracle_attention_us(prefixes, rows_list, parents, n_heads, d):
    """The CPU oracle's tree attention on ONE head of every sequence of the case, scaled to all heads (microseconds)."""
    import oracle
    import synth
    t = 0.0
    for i, (s_, m_, par) in enumerate(zip(prefixes, rows_list, parents)):
        x = synth.qkv(50 + i, 1, d, s_, m_, "bf16")
        t0 = time.perf_counter()
        oracle.tree_attention(x["q"], x["k_prefix"], x["v_prefix"], x["k_tree"], x["v_tree"], par)
        t += time.perf_counter() - t0
    return 1e6 * t * n_heads


def bench_tree_attention(trj, torch, peaks, steps, warmup, cpu=True, only=""):
    """Op-level tree attention on the op-level shapes (configs 2, 4, 5), over distinct caches larger than L2."""
    import synth
    out = []
    h, d = 32, 128
    s5, m5 = synth.ragged_batch(4, 8, (256, 4096), (16, 64))
    cases = (("cfg3 (the step's shape): 32x128 heads, prefix 512, 33-row tree", [512], [33], 6, 3, 16),
             ("cfg2: 32x128 heads, prefix 1024, 64-row tree", [1024], [64], 6, 3, 32),
             ("cfg4: 32x128 heads, prefix 8192, 128-row tree", [8192], [128], 8, 4, 4),
             ("cfg5: 8 sequences, prefix 256-4096, 16-64-row trees", s5.tolist(), m5.tolist(), 6, 3, 2))
    for name, prefixes, rows_list, depth, kids, n_caches in cases:
        if only and only not in name:
            continue
        nb, rows_total = len(prefixes), sum(rows_list)
        max_seq = max(s + m for s, m in zip(prefixes, rows_list))
        g = torch.Generator(device="cuda"); g.manual_seed(7)
        rnd = lambda *shape: torch.randn(*shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        k, v, q = rnd(n_caches, nb, h, max_seq, d), rnd(n_caches, nb, h, max_seq, d), rnd(n_caches, rows_total, h, d)
        o = torch.empty_like(q)
        parents = [synth.random_tree(1 + i, m, min(depth, m - 1), kids) for i, m in enumerate(rows_list)]
        anc = np.concatenate([trj.tree_from_parents(par)[1] for par in parents], 0)
        anc_d = torch.from_numpy(anc.view(np.int64)).cuda()
        seq_len = torch.tensor(prefixes, dtype=torch.int32, device="cuda")
        row_off = torch.tensor(np.concatenate([[0], np.cumsum(rows_list)]), dtype=torch.int32, device="cuda")
        ws = torch.zeros(max(256, trj.tree_attention_workspace(rows_total, nb, h, d, max_seq)), dtype=torch.uint8, device="cuda")

        def one_pass():
            for c in range(n_caches):
                trj.tree_attention(q[c], k[c], v[c], seq_len, row_off, anc_d, max_rows=max(rows_list), max_len=max_seq,
                                   out=o[c], workspace=ws)
        us = graph_us(torch, one_pass, steps, warmup) / n_caches
        nbytes = sum(2 * h * (s + m) * d * 2 for s, m in zip(prefixes, rows_list)) + 2 * rows_total * h * d * 2
        gbs = nbytes / us / 1e3
        out.append({"workload": name, "us_per_launch": round(us, 2), "algorithmic_bytes": nbytes, "hbm_gbs": round(gbs, 1),
                    "frac_of_" + peaks["source"] + "_peak": round(gbs / peaks["hbm_gbs"], 4),
                    "distinct_caches": n_caches})
        if cpu:
            out[-1]["cpu_oracle_us"] = round(oracle_attention_us(prefixes, rows_list, parents, h, d), 1)
            out[-1]["cpu_oracle_sample"] = "one head per sequence, timed once, x %d heads" % h
        del k, v, q, o
    return out


def bench_small_ops(trj, torch, peaks, steps, warmup, cpu=True):
    """Arg-max + acceptance on the 64 x 32000 logits of config 2 and KV compaction of a 7B-shaped cache."""
    import synth
    out = []
    # arg-max + accept: 32 distinct bf16 logit arrays (131 MB in total, larger than L2)
    rows, vocab, n_arr = 64, 32000, 32
    g = torch.Generator(device="cuda"); g.manual_seed(11)
    logits = torch.randn(n_arr, rows, vocab, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    parent = synth.random_tree(1, rows, 6, 3)
    depth, _ = trj.tree_from_parents(parent)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    tokens, d_parent, d_depth, off = i32(synth.prompt(3, rows, vocab)), i32(parent), i32(depth), i32([0, rows])
    outs = {"node_argmax": torch.empty(rows, dtype=torch.int32, device="cuda"), "margin": None,
            "k_acc": torch.empty(1, dtype=torch.int32, device="cuda"), "bonus": torch.empty(1, dtype=torch.int32, device="cuda"),
            "path": torch.empty(1, trj.PATH_STRIDE, dtype=torch.int32, device="cuda")}
    nbytes = rows * vocab * 2
    ws = torch.zeros(trj.argmax_accept_workspace(rows, 1), dtype=torch.uint8, device="cuda")

    def argmax_pass():                                       # the entry point the verification step itself uses
        for a in range(n_arr):
            trj.argmax_accept_into(logits[a], tokens, d_parent, d_depth, off, outs, ws)
    us = graph_us(torch, argmax_pass, steps, warmup) / n_arr
    out.append({"op": "argmax_accept, 64 x 32000 bf16 logits (cfg2)", "us_per_launch": round(us, 2),
                "algorithmic_bytes": nbytes, "hbm_gbs": round(nbytes / us / 1e3, 1),
                "frac_of_" + peaks["source"] + "_peak": round(nbytes / us / 1e3 / peaks["hbm_gbs"], 4)})
    if cpu:
        import oracle
        lg = logits[0].float().cpu().numpy()
        t0 = time.perf_counter()
        pr = oracle.node_argmax(lg)
        oracle.accept_path(tokens.cpu().numpy(), parent, pr)
        out[-1]["cpu_oracle_us"] = round(1e6 * (time.perf_counter() - t0), 1)
    trj.argmax_accept_static(logits[0], tokens, d_parent, d_depth, off, outs)      # one-time set-up outside the capture
    torch.cuda.synchronize()

    def argmax_static_pass():                                # the workspace-free variant: one more memset node per call
        for a in range(n_arr):
            trj.argmax_accept_static(logits[a], tokens, d_parent, d_depth, off, outs)
    us = graph_us(torch, argmax_static_pass, steps, warmup) / n_arr
    out.append({"op": "argmax_accept_static (library-held scratch), same input", "us_per_launch": round(us, 2),
                "algorithmic_bytes": nbytes, "hbm_gbs": round(nbytes / us / 1e3, 1)})
    tk_ws = torch.zeros(trj.lib().trj_topk_accept_workspace(), dtype=torch.uint8, device="cuda")

    def topk_pass():                                         # per-row top-10 + acceptance (templates with top-K siblings)
        for a in range(n_arr):
            trj.topk_accept(logits[a], tokens, d_parent, d_depth, off, 10, workspace=tk_ws)
    us = graph_us(torch, topk_pass, steps, warmup) / n_arr
    out.append({"op": "topk_accept K = 10, same input", "us_per_launch": round(us, 2), "algorithmic_bytes": nbytes,
                "hbm_gbs": round(nbytes / us / 1e3, 1), "frac_of_" + peaks["source"] + "_peak": round(nbytes / us / 1e3 / peaks["hbm_gbs"], 4)})
    del logits
    # compaction: 32 layers x 32 heads x 128, k = 4 accepted rows of a 33-row tree behind a 512-row prefix
    n_layers, h, d, max_seq, k_acc = 32, 32, 128, 640, 4
    kc = torch.zeros(n_layers, 1, h, max_seq, d, dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    seq0 = torch.tensor([512], dtype=torch.int32, device="cuda")
    seq = seq0.clone()
    path = torch.full((1, trj.PATH_STRIDE), -1, dtype=torch.int32, device="cuda")
    path[0, :5] = torch.tensor([0, 6, 7, 8, 9], dtype=torch.int32)
    kk = torch.tensor([k_acc], dtype=torch.int32, device="cuda")

    def compact_pass():
        seq.copy_(seq0)
        trj.compact_rows(kc, vc, seq, kk, path)
    us = graph_us(torch, compact_pass, steps, warmup)
    nbytes = 2 * 2 * k_acc * n_layers * h * d * 2                       # K and V, read + write
    out.append({"op": "compact_rows, 7B cache, k = 4", "us_per_launch": round(us, 2), "algorithmic_bytes": nbytes,
                "hbm_gbs": round(nbytes / us / 1e3, 1),
                "frac_of_" + peaks["source"] + "_peak": round(nbytes / us / 1e3 / peaks["hbm_gbs"], 4)})
    if cpu:
        import oracle
        host = np.zeros((n_layers, h, max_seq, d), np.float32)
        t0 = time.perf_counter()
        oracle.compact_rows(host, 512, [0, 6, 7, 8, 9])
        oracle.compact_rows(host, 512, [0, 6, 7, 8, 9])      # K and V
        out[-1]["cpu_oracle_us"] = round(1e6 * (time.perf_counter() - t0), 1)
    return out


def run_ops_only(args):
    """The op-level legs alone (no model): one JSON line, not the bench contract's."""
    import torch
    import paper_2406_17404_b200 as trj
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verification step has no CPU path")
    torch.cuda.set_device(0)
    trj.lib()
    peaks = measured_peaks()
    steps = max(args.steps, 5)
    out = {"ops_only": True}
    if args.case == "" or args.case.startswith("cfg"):       # "cfg" alone: every attention case
        out["tree_attention"] = bench_tree_attention(trj, torch, peaks, steps, 3, cpu=False, only=args.case)
    if args.case in ("", "small"):
        out["small_ops"] = bench_small_ops(trj, torch, peaks, steps, 3, cpu=False)
    if args.case in ("", "gemm"):
        out["prefill_gemm"] = bench_prefill_gemm(trj, torch, peaks, steps)
    print(json.dumps(out), flush=True)


def run_profile_step(args):
    """A short, fixed launch sequence for a profiler: model set-up, prefill of the prompt, then `--steps` verification
    steps (forward, arg-max + accept, compaction) launched one by one, without a CUDA graph.  Prints the number of
    library launches before the first step and per step, so that a capture can skip to the steps."""
    import torch
    import synth
    from synth.device import device_weights
    import paper_2406_17404_b200 as trj
    trj.lib()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cfg = synth.LLAMA7B if not args.layers else synth.LLAMA7B.with_layers(args.layers)
    layers, glob = device_weights(cfg, 1234, dev)
    model = trj.Model(cfg, layers, glob, max_batch=1, max_seq=PROMPT + 256, max_rows=trj.MAX_ROWS)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    prompt = synth.prompt(100, PROMPT, cfg.vocab)
    first = model.prefill(i32(prompt))
    ctx = np.concatenate([prompt, [int(first.item())]]).astype(np.int32)
    draws = np.asarray(synth.noise_draws(0, 1, WIDTH + N_BRANCHES * BRANCH_LEN), np.int64)
    window = ctx[np.asarray(synth.noise_draws(0, 0, WIDTH), np.int64) % len(ctx)]
    tree = trj.build_tree(int(ctx[-1]), window, trj.retrieve(ctx, N_BRANCHES, BRANCH_LEN, draws[WIDTH:]))
    d_tok, d_par, d_dep, d_off = i32(tree["tokens"]), i32(tree["parent"]), i32(tree["depth"]), i32([0, TREE_ROWS])
    d_anc = torch.from_numpy(tree["anc"].view(np.int64)).to(dev)
    seq0 = model.seq_len.clone()
    torch.cuda.synchronize()
    before = trj.launch_count()
    for _ in range(args.steps):
        model.seq_len.copy_(seq0)
        out = model.verify_step(d_tok, d_par, d_dep, d_anc, d_off, max_rows=TREE_ROWS, max_len=PROMPT + TREE_ROWS)
        acc = model.accept(d_tok, d_par, d_dep, d_off, out["node_argmax"])
        model.compact_kv(acc["k_acc"], acc["path"])
    torch.cuda.synchronize()
    print(json.dumps({"profile_step": True, "layers": cfg.n_layers, "library_launches_before_the_steps": before,
                      "library_launches_per_step": (trj.launch_count() - before) // max(args.steps, 1)}), flush=True)
    model.close()


def oracle_step_inputs(cfg, seed):
    """A verification step's inputs for the CPU oracle: a 33-row tree and a 512-row cache of N(0,1) K/V rows."""
    import oracle
    import synth
    window = synth.prompt(seed + 1, WIDTH, cfg.vocab)
    branches = synth.prompt(seed + 2, N_BRANCHES * BRANCH_LEN, cfg.vocab).reshape(N_BRANCHES, BRANCH_LEN)
    return oracle.build_tree(17, window, branches)


def fill_cache(dec, seed):
    import synth
    cache = dec.new_cache(PROMPT + TREE_ROWS)
    g = synth.stream(seed, "oracle_cache")
    cache.k[:, :, :PROMPT] = g.standard_normal(cache.k[:, :, :PROMPT].shape)
    cache.v[:, :, :PROMPT] = g.standard_normal(cache.v[:, :, :PROMPT].shape)
    cache.seq_len = PROMPT
    return cache


def oracle_sample_model(cfg_full, seed=0):
    """A 2-layer slice of the 7B shape for the CPU oracle (weights drawn once, on the host)."""
    import oracle
    import synth
    cfg = cfg_full.with_layers(2)
    layers = [synth.layer_weights(cfg, seed, l) for l in range(2)]
    return oracle.Decoder(cfg, layers, synth.global_weights(cfg, seed))


def oracle_sample(dec, seed=0):
    """The CPU oracle on a bounded sample of the workload: one verification step of a 2-layer slice of the 7B shape
    (33 rows over a 512-row cache) plus the LM head.  Returns (measured seconds of the sample, seconds of the LM
    head alone) so that the caller can state measurement and extrapolation separately."""
    from oracle.model import rmsnorm, verify_step
    cfg, glob = dec.cfg, dec.glob
    cache = fill_cache(dec, seed)
    tokens, parent = oracle_step_inputs(cfg, seed)
    # the LM head on its own, so that only the layer part is scaled
    x = np.asarray(glob["embed"], np.float64)[tokens]
    t0 = time.perf_counter()
    _ = rmsnorm(x, np.asarray(glob["final_norm"], np.float64), cfg.rms_eps) @ np.asarray(glob["lm_head"], np.float64).T
    t_head = time.perf_counter() - t0
    t0 = time.perf_counter()
    verify_step(dec, cache, tokens, parent)
    return time.perf_counter() - t0, t_head


class TimedLayers:
    """Per-layer weights for the oracle that records how long fetching them took (not CPU work of the method)."""

    def __init__(self, inner):
        self.inner, self.seconds = inner, 0.0

    def __getitem__(self, l):
        t0 = time.perf_counter()
        w = self.inner[l]
        self.seconds += time.perf_counter() - t0
        return w


def oracle_full_step(cfg, layer_view, glob):
    """ONE real verification step of the whole model by the CPU oracle (all layers, 33 rows, 512-row cache); the
    weights come from the device layer by layer and the time spent fetching them is taken out."""
    import oracle
    from oracle.model import verify_step
    timed = TimedLayers(layer_view)
    dec = oracle.Decoder(cfg, timed, glob)
    cache = fill_cache(dec, 0)
    tokens, parent = oracle_step_inputs(cfg, 0)
    t0 = time.perf_counter()
    verify_step(dec, cache, tokens, parent)
    total = time.perf_counter() - t0
    cpu_s = total - timed.seconds
    return {"value": DRAFTS / cpu_s, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
            "sample": "one full verification step (%d layers, 33 rows, 512-row cache), timed once; fetching the weights "
                      "from the device is excluded" % cfg.n_layers,
            "s_per_step": round(cpu_s, 2), "weight_fetch_s": round(timed.seconds, 2)}


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle, as it stands, on the host cores.  Each timed step is a bounded sample of the
    workload (2 of the 32 layers + the LM head, about a second); `ms_per_step` is the measured time of that sample and
    `value` is the whole-step rate it extrapolates to (layer part x 16), the two stated separately."""
    if rank != 0:
        return
    import synth
    cfg = synth.LLAMA7B
    samples, heads = [], []
    dec = oracle_sample_model(cfg)
    for i in range(args.warmup + args.steps):
        t, th = oracle_sample(dec, seed=i)
        if i >= args.warmup:
            samples.append(t); heads.append(th)
    sample_s, head_s = sum(samples) / len(samples), sum(heads) / len(heads)
    full_s = max(sample_s - head_s, 0.0) * cfg.n_layers / 2 + head_s
    val = DRAFTS / full_s
    cores = cpu_threads()
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sample_s, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg, "cpu oracle"),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "per timed step: one verification step of layers 0-1 of 32 plus the LM head (33 rows, "
                                       "512-row cache), measured; value = 32 drafts / (layer part x 16 + LM head)",
                             "measured_sample_s": round(sample_s, 4), "lm_head_s": round(head_s, 4),
                             "layers_in_sample": 2, "layers_full": cfg.n_layers, "extrapolated_full_step_s": round(full_s, 3)},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def workload_config(cfg, l2_note):
    return {"workload": "configs[2]: LLaMA-2-7B-shaped random-init decoder, bf16, prompt 512, TR-Jacobi trees of 32 "
                        "draft tokens + root (window 5 + 9 retrieved branches of 3); one full verification step",
            "n_layers": cfg.n_layers, "d_model": cfg.d_model, "n_heads": cfg.n_heads, "head_dim": cfg.head_dim,
            "d_ff": cfg.d_ff, "vocab": cfg.vocab, "tree_rows": TREE_ROWS, "draft_tokens_per_step": DRAFTS,
            "prefix": PROMPT, "batch": 1, "parallelism": "replicas", "l2": l2_note}


def aggregate_over_ranks(ms_total, e2e_s, launches, world, device):
    """Replicas only: the job takes as long as its slowest rank (MAX of the times) and launches add up."""
    if world <= 1:
        return ms_total, e2e_s, launches
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_total, e2e_s], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([launches], dtype=torch.int64, device=device)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), int(n[0])


def whole_job_rate(world, units_per_rank, seconds):
    """Units all ranks processed divided by the (max-over-ranks) time: every replica does the same work."""
    return world * units_per_rank / seconds


def bench_template_step(trj, torch, synth, model, cfg, prefix, side, steps, context=None, truth=None, take=None):
    """One verification step over a 69-row static template with top-K siblings (63 draft nodes + a retrieval path of
    5 + the root: the tree size the paper uses, Appendix B; the topology is a seeded stand-in): forward, per-row top-10,
    acceptance and compaction, replayed from a CUDA graph on the same model and cache."""
    dev = model.device
    parent, rank = synth.tree_template(0)
    m = len(parent)
    depth, anc = trj.tree_from_parents(parent)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    d_tok, d_par, d_dep, d_off = i32(synth.prompt(77, m, cfg.vocab)), i32(parent), i32(depth), i32([0, m])
    d_anc = torch.from_numpy(anc.view(np.int64)).to(dev)
    pred = torch.empty(m, dtype=torch.int32, device=dev)
    topk = torch.empty(m, 10, dtype=torch.int32, device=dev)
    acc = {"k_acc": torch.empty(1, dtype=torch.int32, device=dev), "bonus": torch.empty(1, dtype=torch.int32, device=dev),
           "path": torch.empty(1, trj.PATH_STRIDE, dtype=torch.int32, device=dev)}
    seq0 = torch.full_like(model.seq_len, prefix)

    def step():
        model.seq_len.copy_(seq0)
        model.verify_step(d_tok, d_par, d_dep, d_anc, d_off, max_rows=m, max_len=prefix + m, node_argmax=pred)
        model.node_topk(m, 10, out=topk)
        model.accept(d_tok, d_par, d_dep, d_off, pred, out=acc)
        model.compact_kv(acc["k_acc"], acc["path"])
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        step()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    out = {"tree_rows": m, "draft_tokens_per_step": m - 1, "top_k": 10, "ms_per_step": ms,
           "draft_tokens_verified_per_s": (m - 1) / (ms / 1e3),
           "what": "7B shape, prefix %d, 63-node template + retrieval path of 5 + root; random drafts" % prefix}
    if context is not None:
        # the whole loop on the device (tokens of the tree, retrieval, forward, top-K + acceptance, compaction, commit
        # and refill from the top-K table): `steps` steps enqueued at once from the prompt's state, wall clock incl.
        # the upload of the draws and the read-back of the committed tokens
        n_retr = int((rank < 0).sum())
        n0 = len(context)
        per_step = int(depth.max()) + 1
        draw = lambda st, n: synth.noise_draws(99, st, n)
        host_ctx = np.zeros(n0 + steps * per_step, np.int32); host_ctx[:n0] = context
        host_drafts = np.asarray(context, np.int32)[np.asarray(draw(0, m - 1), np.int64) % n0]
        host_draws = np.stack([np.asarray(draw(st, m - 1 + n_retr), np.int64) for st in range(1, steps + 1)])
        k_log = torch.zeros(steps, dtype=torch.int32, device=dev)
        if truth is not None:                                # the true continuation planted into the retrieval path, 0-3 tokens a step
            model.set_draft_source(i32(truth), i32(np.asarray(take[:steps], np.int32)))

        def loop():
            model.seq_len.copy_(seq0)
            d_ctx, d_n = i32(host_ctx), i32([n0])
            d_drafts = i32(host_drafts)
            d_draws = torch.from_numpy(host_draws).to(dev)
            model.decode_device_tree(d_ctx, d_n, n0, parent, rank, 10, n_retr, d_drafts, d_draws, steps, k_log=k_log)
            return d_ctx.cpu(), int(d_n.item())
        loop()                                               # captures the step's graph
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        tokens_out, n_end = loop()
        wall = time.perf_counter() - t0
        model.device_status()
        model.set_draft_source(None)
        out["device_loop"] = {"ms_per_step": wall / steps * 1e3, "tokens_committed_per_step": (n_end - n0) / steps,
                              "committed_tokens_per_s": (n_end - n0) / wall,
                              "what": "trj_decode_device_tree: %d steps enqueued at once; the true continuation planted "
                                      "into 0-3 slots of the retrieval path per step" % steps}
        if truth is not None:
            out["device_loop"]["matches_autoregressive"] = bool((tokens_out.numpy()[:n_end] == np.asarray(truth)[:n_end]).all())
    return out


def bench_llama3_step(trj, torch, synth, peaks, steps):
    """The same verification step on the shape of the paper's main model family (Table 2): LLaMA-3-8B, grouped-query
    attention with 8 K/V heads, 128 256-way vocabulary; 33-row trees behind a 512-token prompt, random drafts."""
    from synth.device import device_weights
    dev = torch.device("cuda", torch.cuda.current_device())
    cfg = synth.LLAMA3_8B
    layers, glob = device_weights(cfg, 4242, dev)
    model = trj.Model(cfg, layers, glob, max_batch=1, max_seq=PROMPT + 256, max_rows=trj.MAX_ROWS)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    model.prefill(i32(synth.prompt(5, PROMPT, cfg.vocab)))
    tree = trj.build_tree(17, synth.prompt(6, WIDTH, cfg.vocab), synth.prompt(7, N_BRANCHES * BRANCH_LEN, cfg.vocab).reshape(N_BRANCHES, BRANCH_LEN))
    d_tok, d_par, d_dep, d_off = i32(tree["tokens"]), i32(tree["parent"]), i32(tree["depth"]), i32([0, TREE_ROWS])
    d_anc = torch.from_numpy(tree["anc"].view(np.int64)).to(dev)
    seq0 = model.seq_len.clone()
    pred = torch.empty(TREE_ROWS, dtype=torch.int32, device=dev)
    acc = {"k_acc": torch.empty(1, dtype=torch.int32, device=dev), "bonus": torch.empty(1, dtype=torch.int32, device=dev),
           "path": torch.empty(1, trj.PATH_STRIDE, dtype=torch.int32, device=dev)}

    def step():
        model.seq_len.copy_(seq0)
        model.verify_step(d_tok, d_par, d_dep, d_anc, d_off, max_rows=TREE_ROWS, max_len=PROMPT + TREE_ROWS, node_argmax=pred)
        model.accept(d_tok, d_par, d_dep, d_off, pred, out=acc)
        model.compact_kv(acc["k_acc"], acc["path"])
    us = graph_us(torch, step, steps, 3)
    model.device_status()
    hd, kvd, d, f, v = cfg.n_heads * cfg.head_dim, cfg.kv_heads * cfg.head_dim, cfg.d_model, cfg.d_ff, cfg.vocab
    weight_bytes = 2 * (cfg.n_layers * ((hd + 2 * kvd) * d + d * hd + 2 * f * d + d * f) + v * d)
    model.close()
    del layers, glob
    torch.cuda.empty_cache()
    return {"model": "LLaMA-3-8B shape (32 query / 8 K/V heads, d_ff 14336, vocabulary 128256), random init", "tree_rows": TREE_ROWS,
            "prefix": PROMPT, "ms_per_step": us / 1e3, "draft_tokens_verified_per_s": DRAFTS / (us / 1e6),
            "weight_bytes_per_step": weight_bytes, "weight_stream_gbs": round(weight_bytes / us / 1e3, 1),
            "frac_of_" + peaks["source"] + "_peak_whole_step": round(weight_bytes / us / 1e3 / peaks["hbm_gbs"], 4)}


def bench_tp_rank(trj, torch, synth, peaks, steps):
    """One rank's share of the 7B step when heads and feed-forward columns are split over 2, 4 or 8 ranks: every
    segment, the arg-max, acceptance and compaction of a rank's slice, on this one GPU and WITHOUT the sums over
    ranks that come between the segments (64 all-reduces of rows x d_model fp32 per step).  A lower bound on the
    step time of a tensor-parallel job, not a measurement of one."""
    from paper_2406_17404_b200 import tp
    from synth.device import device_weights
    dev = torch.device("cuda", torch.cuda.current_device())
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    full = synth.LLAMA7B
    tree = trj.build_tree(17, synth.prompt(6, WIDTH, full.vocab), synth.prompt(7, N_BRANCHES * BRANCH_LEN, full.vocab).reshape(N_BRANCHES, BRANCH_LEN))
    d_tok, d_par, d_dep, d_off = i32(tree["tokens"]), i32(tree["parent"]), i32(tree["depth"]), i32([0, TREE_ROWS])
    d_anc = torch.from_numpy(tree["anc"].view(np.int64)).to(dev)
    out = {"exchange_bytes": TREE_ROWS * full.d_model * 4, "exchanges_per_step": 2 * full.n_layers, "ranks": {}}
    for world in (2, 4, 8):
        cfg = tp.shard_cfg(full, world)
        layers, glob = device_weights(cfg, 777 + world, dev)       # a slice has the shape of a narrower model
        model = trj.Model(cfg, layers, glob, max_batch=1, max_seq=PROMPT + 256, max_rows=trj.MAX_ROWS)
        model.prefill(i32(synth.prompt(5, PROMPT, cfg.vocab)))
        seq0 = model.seq_len.clone()
        acc = {"k_acc": torch.empty(1, dtype=torch.int32, device=dev), "bonus": torch.empty(1, dtype=torch.int32, device=dev),
               "path": torch.empty(1, trj.PATH_STRIDE, dtype=torch.int32, device=dev)}

        def step():
            model.seq_len.copy_(seq0)
            model.tp_begin(d_tok, d_par, d_dep, d_anc, d_off, max_rows=TREE_ROWS, max_len=PROMPT + TREE_ROWS)
            for sgm in range(model.tp_segments()):
                model.tp_segment(sgm)
            res = model.tp_finish()
            model.accept(d_tok, d_par, d_dep, d_off, res["node_argmax"], out=acc)
            model.compact_kv(acc["k_acc"], acc["path"])
        us = graph_us(torch, step, steps, 3)
        model.device_status()
        hd, d, f, v = cfg.n_heads * cfg.head_dim, cfg.d_model, cfg.d_ff, cfg.vocab
        weight_bytes = 2 * (cfg.n_layers * (3 * hd * d + d * hd + 2 * f * d + d * f) + v * d)
        out["ranks"][str(world)] = {"ms_per_step_without_exchange": us / 1e3, "weight_bytes_per_rank": weight_bytes,
                                    "weight_stream_gbs": round(weight_bytes / us / 1e3, 1),
                                    "frac_of_" + peaks["source"] + "_peak": round(weight_bytes / us / 1e3 / peaks["hbm_gbs"], 4)}
        model.close()
        del layers, glob, model
        torch.cuda.empty_cache()
    return out


def bench_step_vs_rows(trj, torch, synth, model, cfg, prefix, steps):
    """Verification step (forward + arg-max + acceptance + compaction) against the number of tree rows, on the same
    model and cache: the projections stay weight-bound, so rows are cheap until the accumulators outgrow two CTAs per SM."""
    dev = model.device
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    seq0 = torch.full_like(model.seq_len, prefix)
    out = {}
    for m in (17, 33, 48, 64, 69, 80, 96, 128):
        parent = synth.random_tree(3, m, min(8, m - 1), 4)
        depth, anc = trj.tree_from_parents(parent)
        d_tok, d_par, d_dep, d_off = i32(synth.prompt(77, m, cfg.vocab)), i32(parent), i32(depth), i32([0, m])
        d_anc = torch.from_numpy(anc.view(np.int64)).to(dev)
        pred = torch.empty(m, dtype=torch.int32, device=dev)
        acc = {"k_acc": torch.empty(1, dtype=torch.int32, device=dev), "bonus": torch.empty(1, dtype=torch.int32, device=dev),
               "path": torch.empty(1, trj.PATH_STRIDE, dtype=torch.int32, device=dev)}

        def step():
            model.seq_len.copy_(seq0)
            model.verify_step(d_tok, d_par, d_dep, d_anc, d_off, max_rows=m, max_len=prefix + m, node_argmax=pred)
            model.accept(d_tok, d_par, d_dep, d_off, pred, out=acc)
            model.compact_kv(acc["k_acc"], acc["path"])
        out[str(m)] = round(graph_us(torch, step, steps, 3) / 1e3, 4)
    model.device_status()
    return {"ms_per_step_by_tree_rows": out, "prefix": prefix, "what": "7B shape, random trees and drafts"}


def bench_batched_step(trj, torch, synth, cfg, layers, glob, peaks, steps, n_seq=8):
    """The same verification step for `n_seq` independent sequences at once (each a 512-token prompt and a 33-row
    tree): one forward over all rows, arg-max + acceptance per sequence, compaction of every cache.  The weights are
    streamed once for all sequences, so this is the throughput side of the same kernels; not the headline metric."""
    dev = torch.device("cuda", torch.cuda.current_device())
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    model = trj.Model(cfg, layers, glob, max_batch=n_seq, max_seq=PROMPT + 64, max_rows=TREE_ROWS)
    for b in range(n_seq):
        model.prefill(i32(synth.prompt(300 + b, PROMPT, cfg.vocab)), b)
    trees = [trj.build_tree(17 + b, synth.prompt(400 + b, WIDTH, cfg.vocab),
                            synth.prompt(500 + b, N_BRANCHES * BRANCH_LEN, cfg.vocab).reshape(N_BRANCHES, BRANCH_LEN)) for b in range(n_seq)]
    cat = lambda k: np.concatenate([t[k] for t in trees])
    d_tok, d_par, d_dep = i32(cat("tokens")), i32(cat("parent")), i32(cat("depth"))
    d_anc = torch.from_numpy(np.concatenate([t["anc"] for t in trees], 0).view(np.int64)).to(dev)
    d_off = i32(np.arange(n_seq + 1) * TREE_ROWS)
    rows = n_seq * TREE_ROWS
    seq0 = model.seq_len.clone()
    pred = torch.empty(rows, dtype=torch.int32, device=dev)
    acc = {"k_acc": torch.empty(n_seq, dtype=torch.int32, device=dev), "bonus": torch.empty(n_seq, dtype=torch.int32, device=dev),
           "path": torch.empty(n_seq, trj.PATH_STRIDE, dtype=torch.int32, device=dev)}

    def step():
        model.seq_len.copy_(seq0)
        model.verify_step(d_tok, d_par, d_dep, d_anc, d_off, max_rows=TREE_ROWS, max_len=PROMPT + TREE_ROWS, node_argmax=pred)
        model.accept(d_tok, d_par, d_dep, d_off, pred, out=acc)
        model.compact_kv(acc["k_acc"], acc["path"], batch=n_seq)
    us = graph_us(torch, step, steps, 3)
    model.device_status()
    model.close()
    return {"sequences": n_seq, "tree_rows_each": TREE_ROWS, "prefix": PROMPT, "ms_per_step": us / 1e3,
            "draft_tokens_verified_per_s": n_seq * DRAFTS / (us / 1e6),
            "what": "%d independent sequences in one step (7B shape); random drafts" % n_seq}


def bench_prefill_gemm(trj, torch, peaks, steps):
    """The four projections of the 7B shape on prompt-sized row counts (the tensor-bound side of the projection
    kernel: 128 x 256 tiles), as a stand-alone op: TFLOP/s against the measured dense bf16 peak."""
    out = []
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    shapes = (("qkv", 12288, 4096), ("o", 4096, 4096), ("gate_up", 22016, 4096), ("down", 4096, 11008))
    for m in (512, 2048):
        for name, n, k in shapes:
            x = torch.randn(m, k, generator=g, device="cuda").to(torch.bfloat16)
            w = (torch.randn(n, k, generator=g, device="cuda") * 0.02).to(torch.bfloat16)
            y = torch.empty(m, n, dtype=torch.float32, device="cuda")
            ws = torch.zeros(trj.lib().trj_gemm_workspace(m, n, k), dtype=torch.uint8, device="cuda")
            us = graph_us(torch, lambda: [trj.gemm(x, w, out=y, workspace=ws) for _ in range(4)], steps, 3) / 4
            tf = 2.0 * m * n * k / us / 1e6
            out.append({"shape": "%s: M=%d N=%d K=%d" % (name, m, n, k), "us": round(us, 2), "tflops": round(tf, 1),
                        "frac_of_" + peaks["source"] + "_burst_peak": round(tf / peaks["bf16_tflops"], 4)})
            assert int(ws[:4].view(torch.int32)[0]) == 0
            del x, w, y, ws
    return out


def planted_lengths(seed, n):
    """How many tokens of the true continuation each step's first retrieved branch carries: uniform on 0..3, so
    that a step commits 1 + (0..3) tokens, 2.5 on average (the paper's Table 2 reports 2.0-2.9 per step)."""
    import synth
    return synth.stream(seed, "planted_lengths").integers(0, BRANCH_LEN + 1, size=n).astype(np.int32)


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    import synth
    from synth.device import device_weights, HostView
    import paper_2406_17404_b200 as trj
    from paper_2406_17404_b200 import decode

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verification step has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    trj.lib()
    if args.no_pdl:
        trj.set_pdl(False)
    peaks = measured_peaks()
    cfg = synth.LLAMA7B if not args.layers else synth.LLAMA7B.with_layers(args.layers)
    layers, glob = device_weights(cfg, 1234 + rank, dev)
    warm = max(args.warmup, 3)
    per_step = max(WIDTH, BRANCH_LEN) + 1                    # a step commits at most depth + 1 tokens
    n_host_steps = warm + args.steps                         # the end-to-end loop
    n_loop = args.steps                                      # the device-resident loop (run twice)
    n_truth = per_step * (n_host_steps + 2 * n_loop + 4) + 8
    max_seq = PROMPT + n_truth + TREE_ROWS + 64
    model = trj.Model(cfg, layers, glob, max_batch=1, max_seq=max_seq, max_rows=trj.MAX_ROWS)
    prompt = synth.prompt(100 + rank, PROMPT, cfg.vocab)
    draw = lambda s, n: synth.noise_draws(rank, s, n)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)

    # ---- draft quality.  Random drafts on random weights are never accepted, so every step would commit one token
    # and never move a K/V row.  The true greedy continuation (one-row trees = plain autoregressive decoding, run
    # here before any clock starts) is therefore planted into the first retrieved branch of every step, 0..3 tokens
    # of it, which puts the committed tokens per step at the 2-3 the paper reports.  The same lengths are used by
    # all three timed legs.
    # clock samples run from here (a second or two of the same kernels before the first timed region, so that the
    # sampler is up when it starts) to the end of the device loop
    sampler = ClockSampler(local_rank)
    sampler.start()
    truth = decode.tr_jacobi_generate(model, prompt, n_truth, 0, 0, 0, draw)
    abs_truth = np.concatenate([prompt, np.asarray(truth, np.int32)]).astype(np.int32)     # guess for position i
    take = planted_lengths(rank, n_host_steps + 2 * n_loop + 8)

    def plant(branches, n_ctx, n_take):
        branches = np.array(branches, np.int32, copy=True).reshape(N_BRANCHES, BRANCH_LEN)
        n_take = int(min(n_take, BRANCH_LEN, len(abs_truth) - n_ctx))
        branches[0, :n_take] = abs_truth[n_ctx:n_ctx + n_take]
        return branches

    # ---- state after the prompt
    model.seq_len.zero_()
    first = model.prefill(i32(prompt))
    assert int(first.item()) == truth[0]
    n_ctx0 = PROMPT + 1
    ctx0 = abs_truth[:n_ctx0].copy()
    window0 = ctx0[np.asarray(draw(0, WIDTH), np.int64) % n_ctx0].astype(np.int32)
    s_now = PROMPT                                           # committed cache rows
    seq0 = model.seq_len.clone()

    # ---- timed region 1: inputs resident in HBM.  Four trees (0..3 planted tokens), one CUDA graph each; the timed
    # steps replay them in the order of `take`.  Each replay starts from the same cache state.
    pred = torch.empty(TREE_ROWS, dtype=torch.int32, device=dev)
    acc = {"k_acc": torch.empty(1, dtype=torch.int32, device=dev), "bonus": torch.empty(1, dtype=torch.int32, device=dev),
           "path": torch.empty(1, trj.PATH_STRIDE, dtype=torch.int32, device=dev)}
    d_off = i32([0, TREE_ROWS])
    base_branches = trj.retrieve(ctx0, N_BRANCHES, BRANCH_LEN, np.asarray(draw(1, WIDTH + N_BRANCHES * BRANCH_LEN), np.int64)[WIDTH:])
    side = torch.cuda.Stream(device=dev)
    graphs, k_of, launches_per_step = [], [], 0
    for n_take in range(BRANCH_LEN + 1):
        tree = trj.build_tree(int(ctx0[-1]), window0, plant(base_branches, n_ctx0, n_take))
        d_tok, d_par, d_dep = i32(tree["tokens"]), i32(tree["parent"]), i32(tree["depth"])
        d_anc = torch.from_numpy(tree["anc"].view(np.int64)).to(dev)

        def resident_step(d_tok=d_tok, d_par=d_par, d_dep=d_dep, d_anc=d_anc):
            model.seq_len.copy_(seq0)
            model.verify_step(d_tok, d_par, d_dep, d_anc, d_off, max_rows=TREE_ROWS, max_len=s_now + TREE_ROWS, node_argmax=pred)
            model.accept(d_tok, d_par, d_dep, d_off, pred, out=acc)
            model.compact_kv(acc["k_acc"], acc["path"])
        # the launch sequence of a step is fixed, so it is replayed from a CUDA graph (no host work per launch)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(2):
                resident_step()
        torch.cuda.synchronize()
        k_of.append(int(acc["k_acc"][0]))
        g = torch.cuda.CUDAGraph()
        l0 = trj.launch_count()
        with torch.cuda.graph(g, stream=side):
            resident_step()
        launches_per_step = trj.launch_count() - l0
        graphs.append((g, resident_step))
    for i in range(warm):
        graphs[take[i] % len(graphs)][0].replay()
    torch.cuda.synchronize()
    model.device_status()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        graphs[take[i] % len(graphs)][0].replay()
    e1.record()
    barrier()
    launches = launches_per_step * args.steps
    ms_total = e0.elapsed_time(e1)
    mat_resident = float(np.mean([k_of[take[i] % len(graphs)] + 1 for i in range(args.steps)]))

    # ---- timed region 2: end to end through trj_step_host (host ints in, host result out).  The context lives in
    # one int32 buffer and the random draws the method consumes are inputs: they are generated before the clock starts.
    model.seq_len.copy_(seq0)
    ctx_buf = np.zeros(PROMPT + n_truth + TREE_ROWS, np.int32)
    ctx_buf[:n_ctx0] = ctx0
    n_ctx = n_ctx0
    all_draws = [np.asarray(draw(step, WIDTH + N_BRANCHES * BRANCH_LEN), np.int64) for step in range(n_host_steps + 1)]
    window = window0
    mat = []
    for step in range(1, n_host_steps + 1):
        if step == warm + 1:
            barrier()
            t0 = time.perf_counter()
        draws = all_draws[step]
        context = ctx_buf[:n_ctx]
        branches = plant(trj.retrieve(context, N_BRANCHES, BRANCH_LEN, draws[WIDTH:]), n_ctx, take[step - 1])
        res = model.step_host(int(context[-1]), window, branches, max_len=n_ctx - 1 + TREE_ROWS)
        k = res["k_acc"]
        ctx_buf[n_ctx:n_ctx + k] = res["tokens"][res["path"][1:]]
        ctx_buf[n_ctx + k] = res["bonus"]
        n_ctx += k + 1
        window = trj.refill_window(res["parent"], res["node_argmax"], int(res["path"][-1]), WIDTH, ctx_buf[:n_ctx], draws[:WIDTH])
        mat.append(k + 1)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_matches = bool((ctx_buf[:n_ctx] == abs_truth[:n_ctx]).all())

    # ---- the same loop resident on the device (trj_decode_device): the host uploads the random draws of all steps,
    #      enqueues the steps and reads the generated tokens back at the end; wall clock around all of it
    cap = n_ctx + n_loop * per_step
    host_ctx = np.zeros(cap, np.int32)
    host_ctx[:n_ctx] = ctx_buf[:n_ctx]
    host_ctx_t, host_n_t = torch.from_numpy(host_ctx).pin_memory(), torch.tensor([n_ctx], dtype=torch.int32).pin_memory()
    host_window_t = torch.from_numpy(np.ascontiguousarray(window, dtype=np.int32)).pin_memory()
    loop_draws = torch.from_numpy(np.stack([np.asarray(draw(10_000 + s, WIDTH + N_BRANCHES * BRANCH_LEN), np.int64)
                                            for s in range(n_loop)])).pin_memory()
    d_ctx, d_n = torch.empty(cap, dtype=torch.int32, device=dev), torch.empty(1, dtype=torch.int32, device=dev)
    d_window, d_draws = torch.empty(WIDTH, dtype=torch.int32, device=dev), torch.empty_like(loop_draws, device=dev)
    out_tokens, out_n = torch.empty(cap, dtype=torch.int32).pin_memory(), torch.empty(1, dtype=torch.int32).pin_memory()
    k_log = torch.zeros(n_loop, dtype=torch.int32, device=dev)
    model.set_draft_source(i32(abs_truth), i32(take[n_host_steps:n_host_steps + n_loop]))

    def device_loop():
        t1 = time.perf_counter()
        d_ctx.copy_(host_ctx_t, non_blocking=True); d_n.copy_(host_n_t, non_blocking=True)
        d_window.copy_(host_window_t, non_blocking=True); d_draws.copy_(loop_draws, non_blocking=True)
        model.decode_device(d_ctx, d_n, n_ctx, d_window, N_BRANCHES, BRANCH_LEN, d_draws, n_loop, k_log=k_log)
        out_tokens.copy_(d_ctx, non_blocking=True); out_n.copy_(d_n, non_blocking=True)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t1
        assert int(out_n[0]) - n_ctx >= n_loop
        return dt
    device_loop()                                            # warm-up: same sizes and buffers, so its step graph is reused
    model.seq_len.fill_(n_ctx - 1)                           # rewind the cache to the state before the warm-up loop
    loop_s = device_loop()
    model.set_draft_source(None)
    model.device_status()
    mat_loop = float(k_log.float().mean().item()) + 1.0
    n_end = int(out_n[0])
    loop_matches = bool((out_tokens.numpy()[:n_end] == abs_truth[:n_end]).all())
    loop_h2d = int(host_ctx.nbytes + 4 + host_window_t.numel() * 4 + loop_draws.numel() * 8)
    loop_d2h = int(cap * 4 + 4)
    if world > 1:                                            # replicas: the slowest rank's loop
        t_loop = torch.tensor([loop_s], dtype=torch.float64, device=dev)
        dist.all_reduce(t_loop, op=dist.ReduceOp.MAX)
        loop_s = float(t_loop[0])
    barrier()
    clocks = sampler.stop()

    # ---- per-kernel device time of the same step: a second graph whose launches are bracketed by event
    #      nodes (not part of `value`; the brackets cost a little)
    model.profile_enable(True)
    pgraph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(pgraph, stream=side):
        graphs[2][1]()
    prof = {k: [0.0, 0] for k in trj.PROF_CATEGORIES}
    for i in range(args.steps + 1):
        pgraph.replay()
        torch.cuda.synchronize()
        if i == 0:
            continue                                         # first replay warms the instantiated graph
        for k, (ms, n) in model.profile_read(keep=True).items():
            prof[k][0] += ms
            prof[k][1] += n
    model.profile_enable(False)

    # ---- aggregate over ranks: max time, summed units
    ms_total, e2e_s, launches = aggregate_over_ranks(ms_total, e2e_s, launches, world, dev)
    if rank != 0:
        return
    ms_step = ms_total / args.steps
    value = whole_job_rate(world, DRAFTS * args.steps, ms_total / 1e3)
    e2e_value = whole_job_rate(world, DRAFTS * args.steps, e2e_s)
    mat_e2e = sum(mat[-args.steps:]) / args.steps

    gemm_ms, gemm_launches = prof["gemm"]
    gemm_ms_step = gemm_ms / args.steps
    gbytes = gemm_bytes_per_step(cfg, TREE_ROWS)
    # Inside the replayed step the projections overlap their neighbours (programmatic dependent launch), so their
    # own duration cannot be bracketed without changing it: event nodes around every launch serialise the chain and
    # make the 129 projections alone look longer than the whole real step.  The roofline therefore charges the
    # WHOLE step's device time (timed region 1, CUDA events) to the projections, an upper bound of their duration;
    # the bracketed figure is kept beside it.
    gemm_ms_upper = min(gemm_ms_step, ms_step) if gemm_ms_step > 0 else ms_step
    achieved = gbytes / (gemm_ms_upper / 1e3) / 1e9
    roofline = {"bound": "hbm", "kernel": "projection GEMMs (all %d launches of a step)" % (gemm_launches // args.steps),
                "achieved": achieved, "peak": peaks["hbm_gbs"], "peak_source": peaks["source"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"],
                "traffic": GEMM_TRAFFIC_BYTES_PER_STEP, "algorithmic_bytes_per_step": gbytes,
                "device_ms_per_step": gemm_ms_upper,
                "duration_basis": "whole replayed step (upper bound)" if gemm_ms_upper == ms_step else "event brackets",
                "bracketed_ms_per_step": gemm_ms_step}
    if world == 1 and not args.no_timeline:
        # the projections' own time inside the replayed step, from the clock-stamp build run as a child process
        try:
            child = subprocess.run([sys.executable, os.path.abspath(__file__), "--timeline", "--steps", "5"] +
                                   (["--layers", str(args.layers)] if args.layers else []),
                                   capture_output=True, text=True, timeout=600)
            tl = json.loads(child.stdout.strip().splitlines()[-1])
            roofline["kernel_ms_stamped"] = tl["projection_ms_per_step"]
            roofline["achieved_stamped"] = tl["projection_gbs"]
            roofline["frac_stamped"] = tl["projection_gbs"] / peaks["hbm_gbs"]
            roofline["timeline_per_kernel_us"] = tl["per_kernel_us"]
        except Exception as exc:                             # the headline numbers do not depend on this leg
            roofline["kernel_ms_stamped"] = None
            roofline["timeline_error"] = repr(exc)[:200]
    step_ms_prof = sum(v[0] for v in prof.values()) / args.steps
    breakdown = {k: {"ms_per_step": round(v[0] / args.steps, 4), "launches_per_step": v[1] // args.steps} for k, v in prof.items()}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "verify_step_us": ms_step * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded random weights, prompt and drafts; the true "
            "greedy continuation planted into 0-3 slots of one retrieved branch per step)",
            "config": workload_config(cfg, "13.2 GB of weights per step, far larger than the 126 MB L2"),
            "clocks": clocks, "gpu_launches": launches,
            "tokens_committed_per_step": mat_resident,
            "committed_tokens_per_s": whole_job_rate(world, mat_resident * args.steps, ms_total / 1e3),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": trj.STEP_H2D_BYTES,
                    "d2h_bytes_per_step": trj.STEP_D2H_BYTES, "ms_per_step": 1e3 * e2e_s / args.steps,
                    "tokens_committed_per_step": mat_e2e,
                    "committed_tokens_per_s": whole_job_rate(world, mat_e2e * args.steps, e2e_s),
                    "matches_autoregressive": e2e_matches},
            "device_loop": {"value": whole_job_rate(world, DRAFTS * args.steps, loop_s), "unit": UNIT,
                            "ms_per_step": 1e3 * loop_s / args.steps, "h2d_bytes_total": loop_h2d, "d2h_bytes_total": loop_d2h,
                            "tokens_committed_per_step": mat_loop,
                            "committed_tokens_per_s": whole_job_rate(world, mat_loop * args.steps, loop_s),
                            "matches_autoregressive": loop_matches,
                            "what": "trj_decode_device: %d steps enqueued at once, drafting and refill on the device; "
                                    "wall clock incl. uploading the draws and reading the tokens back" % args.steps},
            "roofline": roofline, "kernel_breakdown": breakdown, "profiled_step_ms": step_ms_prof}
    if world == 1:
        line["paper_sized_tree"] = bench_template_step(trj, torch, synth, model, cfg, PROMPT, side, args.steps, context=ctx0, truth=abs_truth, take=take)
        # prefill of the 512-token prompt: the weights are streamed once (projections over all 512 rows at a time)
        model.seq_len.zero_()
        model.prefill(i32(prompt)); torch.cuda.synchronize()
        pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        model.seq_len.zero_()
        pe0.record(); model.prefill(i32(prompt)); pe1.record(); torch.cuda.synchronize()
        pf_ms = pe0.elapsed_time(pe1)
        pf_flops = 2.0 * PROMPT * (gemm_bytes_per_step(cfg, 0) / 2)        # 2 x rows x weight parameters
        line["prefill"] = {"prompt": PROMPT, "ms": pf_ms, "tflops": pf_flops / pf_ms / 1e9,
                           "note": "projections take bf16-pair activations: two tensor-core products per weight tile"}
        if not args.no_attention:
            line["prefill_gemm"] = bench_prefill_gemm(trj, torch, peaks, max(args.steps // 2, 5))
            line["llama3_8b_step"] = bench_llama3_step(trj, torch, synth, peaks, max(args.steps // 2, 5))
            line["tensor_parallel_rank"] = bench_tp_rank(trj, torch, synth, peaks, max(args.steps // 2, 5))
            line["step_vs_rows"] = bench_step_vs_rows(trj, torch, synth, model, cfg, PROMPT, max(args.steps // 2, 5))
            line["batched_step"] = bench_batched_step(trj, torch, synth, cfg, layers, glob, peaks, max(args.steps // 2, 5))
        if not args.no_attention:
            line["tree_attention"] = bench_tree_attention(trj, torch, peaks, max(args.steps, 5), 3, cpu=not args.no_cpu)
            line["small_ops"] = bench_small_ops(trj, torch, peaks, max(args.steps, 5), 3, cpu=not args.no_cpu)
        if not args.no_cpu:
            line["cpu_baseline"] = oracle_full_step(cfg, HostView(layers), {k: v.float().cpu().numpy() for k, v in glob.items()})
    print(json.dumps(line), flush=True)
    model.close()


def run_timeline(args):
    """Per-kernel clock stamps of the replayed step, from the -DTRJ_TIMELINE build of the library (built here into a
    second shared object; the default library carries no instrumentation).  For every per-layer kernel: the time
    from the moment its first CTA is released by its predecessor to the end of its last CTA, and the gap to the next
    release.  Prints one JSON line; `projection_ms_per_step` is the sum over the 129 projection launches."""
    import torch
    import synth
    from synth.device import device_weights
    from paper_2406_17404_b200 import build as trj_build
    import paper_2406_17404_b200 as trj
    trj.use_library(trj_build.build(timeline=True))
    trj.lib()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    cfg = synth.LLAMA7B if not args.layers else synth.LLAMA7B.with_layers(args.layers)
    layers, glob = device_weights(cfg, 1234, dev)
    model = trj.Model(cfg, layers, glob, max_batch=1, max_seq=PROMPT + 256, max_rows=trj.MAX_ROWS)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    prompt = synth.prompt(100, PROMPT, cfg.vocab)
    first = model.prefill(i32(prompt))
    ctx = np.concatenate([prompt, [int(first.item())]]).astype(np.int32)
    draws = np.asarray(synth.noise_draws(0, 1, WIDTH + N_BRANCHES * BRANCH_LEN), np.int64)
    window = ctx[np.asarray(synth.noise_draws(0, 0, WIDTH), np.int64) % len(ctx)]
    tree = trj.build_tree(int(ctx[-1]), window, trj.retrieve(ctx, N_BRANCHES, BRANCH_LEN, draws[WIDTH:]))
    d_tok, d_par, d_dep, d_off = i32(tree["tokens"]), i32(tree["parent"]), i32(tree["depth"]), i32([0, TREE_ROWS])
    d_anc = torch.from_numpy(tree["anc"].view(np.int64)).to(dev)
    seq0 = model.seq_len.clone()
    pred = torch.empty(TREE_ROWS, dtype=torch.int32, device=dev)
    acc = {"k_acc": torch.empty(1, dtype=torch.int32, device=dev), "bonus": torch.empty(1, dtype=torch.int32, device=dev),
           "path": torch.empty(1, trj.PATH_STRIDE, dtype=torch.int32, device=dev)}

    def step():
        model.seq_len.copy_(seq0)
        trj.timeline_reset()
        model.verify_step(d_tok, d_par, d_dep, d_anc, d_off, max_rows=TREE_ROWS, max_len=PROMPT + TREE_ROWS, node_argmax=pred)
        model.accept(d_tok, d_par, d_dep, d_off, pred, out=acc)
        model.compact_kv(acc["k_acc"], acc["path"])
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(2):
            step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    dur = {k: [] for k in trj.TL_KINDS}
    gap = {k: [] for k in trj.TL_KINDS}
    span, proj, by_proj = [], [], {}
    for _ in range(max(args.steps, 3)):
        graph.replay()
        torch.cuda.synchronize()
        rec = trj.timeline_read()
        events = sorted((int(b), int(e), k) for k, (bs, es) in rec.items() for b, e in zip(bs, es))
        for i, (b, e, k) in enumerate(events):
            dur[k].append((e - b) / 1e3)
            if i + 1 < len(events):
                gap[k].append((events[i + 1][0] - e) / 1e3)
        gemms = [(e - b) / 1e3 for b, e, k in events if k == "gemm"]
        if len(gemms) == 4 * cfg.n_layers + 1:               # QKV, output, gate/up, down per layer, then the LM head
            for i, name in enumerate(("qkv", "o", "gate_up", "down")):
                by_proj.setdefault(name, []).extend(gemms[i:-1:4])
            by_proj.setdefault("lm_head", []).append(gemms[-1])
        span.append((max(e for _, e, _ in events) - min(b for b, _, _ in events)) / 1e6)
        proj.append(sum(e - b for b, e, k in events if k == "gemm") / 1e6)
    mean = lambda v: round(float(np.mean(v)), 3) if v else None
    line = {"timeline": True, "layers": cfg.n_layers, "tree_rows": TREE_ROWS, "prefix": PROMPT,
            "per_kernel_us": {k: {"launches_per_step": len(dur[k]) // max(args.steps, 3), "release_to_end": mean(dur[k]),
                                  "gap_to_next_release": mean(gap[k])} for k in trj.TL_KINDS},
            "projection_us_by_kind": {k: mean(v) for k, v in by_proj.items()},
            "projection_ms_per_step": mean(proj), "first_release_to_last_end_ms": mean(span),
            "projection_ctas_per_sm_peak": trj.timeline_ctas_per_sm(),
            "projection_bytes_per_step": gemm_bytes_per_step(cfg, TREE_ROWS),
            "projection_gbs": round(gemm_bytes_per_step(cfg, TREE_ROWS) / (float(np.mean(proj)) / 1e3) / 1e9, 1)}
    print(json.dumps(line), flush=True)
    model.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="debug: fewer layers than the 7B shape (invalidates the number)")
    ap.add_argument("--no-pdl", action="store_true", help="launch the kernels fully serialised (comparison only)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-timeline", action="store_true", help="skip the clock-stamp leg (a child process with the -DTRJ_TIMELINE build)")
    ap.add_argument("--no-attention", action="store_true", help="skip the op-level tree-attention leg")
    ap.add_argument("--case", default="", help="with --ops-only: cfg | cfg2 | cfg3 | cfg4 | cfg5 | small | gemm (default: all)")
    ap.add_argument("--profile-step", action="store_true",
                    help="prefill + a few un-graphed verification steps and nothing else: a launch sequence for a profiler")
    ap.add_argument("--timeline", action="store_true",
                    help="per-kernel clock stamps of the replayed step from the -DTRJ_TIMELINE build (one JSON line)")
    ap.add_argument("--ops-only", action="store_true",
                    help="only the op-level legs (tree attention, arg-max + accept, compaction): a small run for profiling")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.ops_only:
        if rank == 0:
            run_ops_only(args)
        return
    if args.timeline:
        if rank == 0:
            run_timeline(args)
        return
    if args.profile_step:
        if rank == 0:
            run_profile_step(args)
        return
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if world > 1:
        import torch
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_ours(args, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
