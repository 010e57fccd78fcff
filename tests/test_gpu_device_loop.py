"""GPU parity of device-side drafting, commit/refill and the device-resident decode loop, through the C ABI.

Everything here is integer work: the bar is bit-exact against the oracle's host functions (``oracle.retrieve``,
``oracle.build_tree``, ``oracle.refill_window``) and, for the whole loop, the oracle's greedy TR-Jacobi generation
(committed tokens equal unless an arg-max along the way is decided by less than the margin the parity protocol
excludes).
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import i32
from test_gpu_model import MARGIN, make_models

pytestmark = pytest.mark.gpu


def i64(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int64)).cuda()


def repetitive_context(seed, n, vocab):
    """Tokens over a small vocabulary with copied spans, so that 1- and 2-gram matches are frequent."""
    g = synth.stream(seed, "ctx")
    ctx = g.integers(0, vocab, size=n).astype(np.int32)
    for _ in range(n // 20):
        a, b, ln = (int(x) for x in (g.integers(0, max(n - 8, 1)), g.integers(0, max(n - 8, 1)), g.integers(2, 8)))
        ctx[b:b + ln] = ctx[a:a + ln][:len(ctx[b:b + ln])]
    return ctx


@pytest.mark.parametrize("n,vocab,width,r,lr", [
    (1, 5, 3, 2, 3), (2, 5, 0, 2, 3), (3, 2, 4, 3, 2), (50, 4, 4, 2, 3), (700, 6, 5, 9, 3), (700, 50000, 5, 9, 3),
    (129, 3, 2, 64, 1), (333, 7, 1, 1, 12), (64, 9, 7, 0, 0),
])
def test_draft_tokens_equal_oracle_retrieval_and_tree(trj, n, vocab, width, r, lr):
    for seed in range(4):
        ctx = repetitive_context(seed * 31 + n, n, vocab)
        g = synth.stream(seed, "draws")
        draws = g.integers(0, 2 ** 40, size=width + r * lr).astype(np.int64)
        window = g.integers(0, vocab, size=width).astype(np.int32)
        buf = np.zeros(n + 16, np.int32); buf[:n] = ctx
        got = trj.draft_tokens(i32(buf), i32([n]), i32(window), r, lr, i64(draws)).cpu().numpy()
        branches = oracle.retrieve(ctx.tolist(), r, lr, draws[width:].tolist())
        want, _ = oracle.build_tree(int(ctx[-1]), window.tolist(), branches)
        np.testing.assert_array_equal(got, want)


@pytest.mark.parametrize("m,width", [(1, 3), (11, 4), (33, 5), (64, 8), (128, 2), (20, 0)])
def test_commit_refill_equals_oracle(trj, m, width):
    vocab = 97
    for seed in range(4):
        parent = synth.random_tree(seed + m, m, min(6, max(1, m - 1)), 3) if m > 1 else np.array([-1], np.int32)
        logits = synth.logits(seed, m, vocab, "f32")
        pred = oracle.node_argmax(logits)
        tokens = synth.planted_tokens(seed, parent, pred, vocab, p_hit=0.7)
        k, path, bonus = oracle.accept_path(tokens, parent, pred)
        n = 40 + seed
        ctx = synth.prompt(seed, n, vocab)
        draws = synth.stream(seed, "d").integers(0, 2 ** 40, size=max(width, 1)).astype(np.int64)
        buf = np.zeros(n + m + 4, np.int32); buf[:n] = ctx
        d_ctx, d_n = i32(buf), i32([n])
        path_dev = np.full(trj.PATH_STRIDE, -1, np.int32); path_dev[:k + 1] = path
        window, overflow = trj.commit_refill(i32(tokens), i32(parent), i32(pred), i32([k]), i32(path_dev), i32([bonus]),
                                             d_ctx, d_n, width, i64(draws))
        grown = ctx.tolist() + [int(tokens[r]) for r in path[1:]] + [int(bonus)]
        want = oracle.refill_window(parent.tolist(), pred.tolist(), path[-1], width, grown, draws.tolist())
        assert int(d_n[0]) == len(grown) and int(overflow[0]) == 0
        np.testing.assert_array_equal(d_ctx.cpu().numpy()[:len(grown)], np.asarray(grown, np.int32))
        np.testing.assert_array_equal(window.cpu().numpy(), np.asarray(want, np.int32).reshape(-1))


def test_commit_refill_flags_a_full_context(trj):
    parent = synth.chain_parents(4)
    tokens, pred = i32([7, 8, 9, 10]), i32([8, 9, 10, 11])       # every draft accepted: k = 3
    d_ctx, d_n = i32([1, 2, 3, 0, 0]), i32([3])                  # room for 2 more, 4 are needed
    window, overflow = trj.commit_refill(tokens, i32(parent), pred, i32([3]), i32([0, 1, 2, 3] + [-1] * (trj.PATH_STRIDE - 4)),
                                         i32([11]), d_ctx, d_n, 2, i64([5, 6]))
    assert int(overflow[0]) == 1 and int(d_n[0]) == 3
    assert d_ctx.cpu().tolist() == [1, 2, 3, 0, 0]


def test_device_decode_loop_commits_the_oracle_tokens(trj):
    """Config 1 (tiny fp32 model), 32 steps with no host work in between."""
    cfg = synth.TINY
    model, dec = make_models(trj, cfg, 0, max_seq=64 + 32 * 5 + 16, max_rows=16)
    prompt = synth.prompt(0, 64, cfg.vocab)
    width, r, lr, n_steps = 4, 2, 3, 32
    draw = lambda s, n: synth.noise_draws(0, s, n)
    trace = []
    oracle.tr_jacobi_generate(dec, prompt, 200, width, r, lr, draw, trace=trace)
    trace = trace[:n_steps]
    n_new = sum(rec["k"] + 1 for rec in trace)
    want = oracle.tr_jacobi_generate(dec, prompt, n_new, width, r, lr, draw)

    model.seq_len.zero_()
    first = int(model.prefill(i32(prompt)).item())
    committed = [int(t) for t in prompt] + [first]
    capacity = len(committed) + n_steps * (max(width, lr) + 1)
    buf = np.zeros(capacity, np.int32); buf[:len(committed)] = committed
    d_ctx, d_n = i32(buf), i32([len(committed)])
    window = i32([committed[int(d) % len(committed)] for d in draw(0, width)])
    draws = i64(np.stack([np.asarray(draw(s, width + r * lr), np.int64) for s in range(1, n_steps + 1)]))
    k_log = torch.full((n_steps,), -1, dtype=torch.int32, device="cuda")
    model.decode_device(d_ctx, d_n, len(committed), window, r, lr, draws, n_steps, k_log=k_log)
    torch.cuda.synchronize()
    n_end = int(d_n[0])
    got = d_ctx.cpu().numpy()[len(prompt):n_end].tolist()
    assert int(model.seq_len[0]) == n_end - 1
    assert (k_log.cpu().numpy() >= 0).all() and int(k_log.sum()) + n_steps == n_end - len(committed)
    first_bad = next((i for i, (a, b) in enumerate(zip(got, want)) if a != b), None)
    if first_bad is not None:                              # only a sub-margin arg-max may differ
        ar_margin = min(oracle.top2_margin(rec["logits"]).min() for rec in trace)
        assert ar_margin < MARGIN, f"token {first_bad} differs with all margins >= {MARGIN}"
    else:
        assert k_log.cpu().tolist() == [rec["k"] for rec in trace]
        assert len(got) == n_new + 1                        # the prefill's token, then k + 1 per step
    model.close()


@pytest.mark.parametrize("width,r,lr", [(0, 3, 2), (3, 0, 0), (1, 1, 1)])
def test_device_decode_loop_degenerate_tree_shapes(trj, width, r, lr):
    """No window, no retrieved branches, a single-token window and branch: the loop still commits the oracle's tokens."""
    cfg = synth.TINY
    n_steps = 10
    model, dec = make_models(trj, cfg, 1, max_seq=40 + n_steps * 4 + 16, max_rows=16)
    prompt = synth.prompt(3, 40, cfg.vocab)
    draw = lambda s, n: synth.noise_draws(5, s, n)
    trace = []
    oracle.tr_jacobi_generate(dec, prompt, 60, width, r, lr, draw, trace=trace)
    trace = trace[:n_steps]
    want = oracle.tr_jacobi_generate(dec, prompt, sum(rec["k"] + 1 for rec in trace), width, r, lr, draw)
    model.seq_len.zero_()
    first = int(model.prefill(i32(prompt)).item())
    committed = [int(t) for t in prompt] + [first]
    buf = np.zeros(len(committed) + n_steps * (max(width, lr) + 1), np.int32); buf[:len(committed)] = committed
    d_ctx, d_n = i32(buf), i32([len(committed)])
    window = i32([committed[int(d) % len(committed)] for d in draw(0, width)]) if width else torch.empty(0, dtype=torch.int32, device="cuda")
    per = max(width + r * lr, 1)
    draws = i64(np.stack([np.resize(np.asarray(draw(s, width + r * lr), np.int64), per) for s in range(1, n_steps + 1)]))
    if width + r * lr == 0:
        pytest.skip("a tree of the root alone needs no draws")
    model.decode_device(d_ctx, d_n, len(committed), window, r, lr, draws, n_steps)
    torch.cuda.synchronize()
    got = d_ctx.cpu().numpy()[len(prompt):int(d_n[0])].tolist()
    first_bad = next((i for i, (a, b) in enumerate(zip(got, want)) if a != b), None)
    if first_bad is not None:
        assert min(oracle.top2_margin(rec["logits"]).min() for rec in trace) < MARGIN
    else:
        assert len(got) == len(want) + 1
    model.close()


def test_device_decode_loop_with_an_external_draft_source(trj):
    """Drafts planted from an external source (here: the oracle's own greedy continuation, so they are all correct):
    step s accepts at least take[s] rows, and the loop still commits the oracle's greedy tokens (Eq. 1)."""
    cfg = synth.TINY
    width, r, lr, n_steps = 4, 2, 3, 12
    model, dec = make_models(trj, cfg, 0, max_seq=64 + n_steps * 5 + 32, max_rows=16)
    prompt = synth.prompt(9, 64, cfg.vocab)
    draw = lambda s, n: synth.noise_draws(9, s, n)
    n_truth = n_steps * (max(width, lr) + 1) + 2
    truth = oracle.autoregressive_greedy(dec, prompt, n_truth)
    take_host = np.asarray([s % 4 for s in range(n_steps)], np.int32)            # 0..3 planted tokens per step
    model.seq_len.zero_()
    first = int(model.prefill(i32(prompt)).item())
    assert first == truth[0]
    committed = [int(t) for t in prompt] + [first]
    buf = np.zeros(len(prompt) + n_truth, np.int32); buf[:len(committed)] = committed
    d_ctx, d_n = i32(buf), i32([len(committed)])
    window = i32([committed[int(d) % len(committed)] for d in draw(0, width)])
    draws = i64(np.stack([np.asarray(draw(s, width + r * lr), np.int64) for s in range(1, n_steps + 1)]))
    k_log = torch.full((n_steps,), -1, dtype=torch.int32, device="cuda")
    stream = i32(np.concatenate([prompt, truth]))                                # guess for position i = the true token
    model.set_draft_source(stream, i32(take_host))
    model.decode_device(d_ctx, d_n, len(committed), window, r, lr, draws, n_steps, k_log=k_log)
    torch.cuda.synchronize()
    model.set_draft_source(None)
    n_end = int(d_n[0])
    got = d_ctx.cpu().numpy()[len(prompt):n_end].tolist()
    # margins of the oracle's own run decide whether a difference is admissible
    if got != truth[:len(got)]:
        cache = dec.new_cache(len(prompt) + n_truth + 1)
        lg = dec.forward_rows(cache, list(prompt) + truth[:len(got)], list(range(-1, len(prompt) + len(got) - 1)))
        assert oracle.top2_margin(lg[len(prompt) - 1:]).min() < MARGIN
    else:
        assert (k_log.cpu().numpy() >= np.minimum(take_host, lr)).all()
        assert int(k_log.sum()) + n_steps == n_end - len(committed)
    model.close()


def test_device_template_loop_with_an_external_draft_source(trj):
    """The same source feeding the start of a template's retrieval path: step s accepts at least take[s] rows and the
    loop commits the oracle's greedy tokens."""
    cfg = synth.TINY
    parent, rank = synth.tree_template(0)
    m, top_k, n_retr, n_steps = len(parent), 10, 5, 10
    model, dec = make_models(trj, cfg, 0, max_seq=512, max_rows=128)
    prompt = synth.prompt(9, 64, cfg.vocab)
    draw = lambda s, n: synth.noise_draws(9, s, n)
    per_step = int(synth.node_depths(np.asarray(parent, np.int32)).max()) + 1
    n_truth = n_steps * per_step + 2
    truth = oracle.autoregressive_greedy(dec, prompt, n_truth)
    take_host = np.asarray([s % 4 for s in range(n_steps)], np.int32)
    model.seq_len.zero_()
    first = int(model.prefill(i32(prompt)).item())
    assert first == truth[0]
    committed = [int(t) for t in prompt] + [first]
    buf = np.zeros(len(prompt) + n_truth, np.int32); buf[:len(committed)] = committed
    d_ctx, d_n = i32(buf), i32([len(committed)])
    drafts = i32([committed[int(d) % len(committed)] for d in draw(0, m - 1)])
    draws = i64(np.stack([np.asarray(draw(s, m - 1 + n_retr), np.int64) for s in range(1, n_steps + 1)]))
    k_log = torch.full((n_steps,), -1, dtype=torch.int32, device="cuda")
    model.set_draft_source(i32(np.concatenate([prompt, truth])), i32(take_host))
    model.decode_device_tree(d_ctx, d_n, len(committed), parent, rank, top_k, n_retr, drafts, draws, n_steps, k_log=k_log)
    torch.cuda.synchronize()
    model.set_draft_source(None)
    n_end = int(d_n[0])
    got = d_ctx.cpu().numpy()[len(prompt):n_end].tolist()
    if got != truth[:len(got)]:
        cache = dec.new_cache(len(prompt) + n_truth + 1)
        lg = dec.forward_rows(cache, list(prompt) + truth[:len(got)], list(range(-1, len(prompt) + len(got) - 1)))
        assert oracle.top2_margin(lg[len(prompt) - 1:]).min() < MARGIN
    else:
        assert (k_log.cpu().numpy() >= take_host).all()
        assert int(k_log.sum()) + n_steps == n_end - len(committed)
    model.close()


def test_device_decode_loop_7b_shape_equals_the_host_driven_loop(trj):
    """7B layer shape, 2 layers, bf16 (the tcgen05 kernels): the device-resident loop and the host-driven loop run the
    same kernels on the same inputs, so their committed tokens must be identical.  This checks the loop's plumbing on
    that path; parity of the path itself with the oracle is test_llama7b_shape_two_layers_bf16's job."""
    from paper_2406_17404_b200.decode import tr_jacobi_generate
    cfg = synth.LLAMA7B.with_layers(2)
    model, _ = make_models(trj, cfg, 2, max_seq=256, max_rows=128)
    prompt = synth.prompt(7, 70, cfg.vocab)
    width, r, lr, n_steps = 5, 9, 3, 5
    draw = lambda s, n: synth.noise_draws(3, s, n)
    gtrace = []
    tr_jacobi_generate(model, prompt, n_steps, width, r, lr, draw, trace=gtrace)     # stops after <= n_steps steps
    gtrace = gtrace[:n_steps]
    host_tokens = []
    for rec in gtrace:
        host_tokens += [int(rec["tokens"][i]) for i in rec["path"][1:]] + [int(rec["bonus"])]

    model.seq_len.zero_()
    first = int(model.prefill(i32(prompt)).item())
    committed = [int(t) for t in prompt] + [first]
    steps = len(gtrace)
    buf = np.zeros(len(committed) + steps * (max(width, lr) + 1), np.int32); buf[:len(committed)] = committed
    d_ctx, d_n = i32(buf), i32([len(committed)])
    window = i32([committed[int(d) % len(committed)] for d in draw(0, width)])
    draws = i64(np.stack([np.asarray(draw(s, width + r * lr), np.int64) for s in range(1, steps + 1)]))
    model.decode_device(d_ctx, d_n, len(committed), window, r, lr, draws, steps)
    torch.cuda.synchronize()
    got = d_ctx.cpu().numpy()[len(committed):int(d_n[0])].tolist()
    assert got == host_tokens
    model.close()


def test_device_decode_loop_checks_capacity_on_the_host(trj):
    cfg = synth.TINY
    model, _ = make_models(trj, cfg, 0, max_seq=128, max_rows=16)
    d_ctx, d_n = i32(np.zeros(40, np.int32)), i32([30])
    with pytest.raises(trj.TrjError):                       # 30 + 3 * 5 > 40
        model.decode_device(d_ctx, d_n, 30, i32([1, 2, 3, 4]), 2, 3, i64(np.zeros((3, 10))), 3)
    with pytest.raises(trj.TrjError):                       # 1 + 4 + 6 * 3 rows > max_rows 16
        model.decode_device(i32(np.zeros(400, np.int32)), d_n, 30, i32([1, 2, 3, 4]), 6, 3, i64(np.zeros((1, 22))), 1)
    model.close()


def test_device_template_loop_equals_the_host_driven_loop_and_the_oracle(trj):
    """A 69-row template with top-K siblings and a retrieval path (Appendix B), tiny fp32 model: the loop that stays
    on the device (tokens, forward, top-K + acceptance, compaction, commit + refill from the top-K table) against
    the host-driven loop over the same kernels (bit-exact: accepted counts, context, next drafts) and against the
    oracle's template decoding (equal unless a near-tie fell the other way)."""
    from paper_2406_17404_b200.decode import tr_jacobi_generate_tree
    cfg = synth.TINY
    model, dec = make_models(trj, cfg, 0, max_seq=512, max_rows=128)
    prompt = synth.prompt(0, 64, cfg.vocab)
    parent, rank = synth.tree_template(0)
    m, top_k, n_retr, n_steps = len(parent), 10, 5, 12
    draw = lambda s, n: synth.noise_draws(4, s, n)
    # host-driven loop over the same kernels: its trace gives every step's accepted count and tokens
    gtrace = []
    tr_jacobi_generate_tree(model, prompt, 6 * n_steps, parent, rank, top_k, n_retr, draw, trace=gtrace)   # a step commits at most 6 tokens
    assert len(gtrace) >= n_steps
    gtrace = gtrace[:n_steps]
    # the device loop from the same start
    model.seq_len.zero_()
    first = int(model.prefill(i32(prompt)).item())
    committed = [int(t) for t in prompt] + [first]
    depth = synth.node_depths(np.asarray(parent, np.int32))
    capacity = len(committed) + n_steps * (int(depth.max()) + 1)
    buf = np.zeros(capacity, np.int32); buf[:len(committed)] = committed
    d_ctx, d_n = i32(buf), i32([len(committed)])
    drafts = i32([committed[int(d) % len(committed)] for d in draw(0, m - 1)])
    draws = i64(np.stack([np.asarray(draw(s, m - 1 + n_retr), np.int64) for s in range(1, n_steps + 1)]))
    k_log = torch.full((n_steps,), -1, dtype=torch.int32, device="cuda")
    model.decode_device_tree(d_ctx, d_n, len(committed), parent, rank, top_k, n_retr, drafts, draws, n_steps, k_log=k_log)
    torch.cuda.synchronize()
    model.device_status()
    n_end = int(d_n[0])
    got = d_ctx.cpu().numpy()[:n_end].tolist()
    want_host = list(committed)
    for rec in gtrace:
        want_host += [int(rec["tokens"][r]) for r in rec["path"][1:]] + [rec["bonus"]]
    assert k_log.cpu().tolist() == [rec["k_acc"] for rec in gtrace]
    assert got == want_host
    assert int(model.seq_len[0]) == n_end - 1
    # the drafts left for the next step are what the host refill makes of the last step's top-K table
    last = gtrace[-1]
    retrieved = trj.retrieve(want_host[:len(want_host) - last["k_acc"] - 1], 1, n_retr, np.asarray(draw(n_steps, m - 1 + n_retr), np.int64)[m - 1:])[0]
    want_drafts = trj.refill_tree(parent, rank, last["topk"], int(last["path"][-1]), want_host,
                                  np.asarray(draw(n_steps, m - 1 + n_retr), np.int64)[:m - 1], retrieved)
    np.testing.assert_array_equal(drafts.cpu().numpy(), want_drafts)
    # and the oracle: greedy decoding commits the autoregressive tokens (Eq. 1)
    want = oracle.autoregressive_greedy(dec, prompt, n_end - len(prompt))
    if got[len(prompt):] != want:
        trace = []
        oracle.tr_jacobi_generate_tree(dec, prompt, n_end - len(prompt), parent, rank, top_k, n_retr, draw, trace=trace)
        assert min(oracle.top2_margin(rec["logits"]).min() for rec in trace) < MARGIN
    assert int(k_log.max()) >= 1
    model.close()


def test_device_template_loop_checks_the_template_on_the_host(trj):
    cfg = synth.TINY
    model, _ = make_models(trj, cfg, 0, max_seq=256, max_rows=32)
    d_ctx, d_n = i32(np.zeros(200, np.int32)), i32([10])
    drafts, draws = i32(np.zeros(3, np.int32)), i64(np.zeros((2, 4), np.int64))
    good_parent, good_rank = [-1, 0, 0, 1], [0, 0, 1, -1]
    for parent, rank, k, n_retr in (([-1, 0, 0, 3], good_rank, 2, 1),      # parent is not an earlier row
                                   (good_parent, [0, 0, 2, -1], 2, 1),     # rank >= K
                                   (good_parent, [0, 0, 1, -2], 2, 1),     # retrieval slot past n_retrieved
                                   (good_parent, good_rank, 11, 1)):       # K past the limit
        with pytest.raises(trj.TrjError):
            model.decode_device_tree(d_ctx, d_n, 10, parent, rank, k, n_retr, drafts, draws, 2)
    with pytest.raises(trj.TrjError):                                      # the context buffer cannot take the steps
        model.decode_device_tree(i32(np.zeros(12, np.int32)), d_n, 10, good_parent, good_rank, 2, 1, drafts, draws, 2)
    torch.cuda.synchronize()
    model.close()
