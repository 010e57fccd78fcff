"""The workspace-free arg-max + accept entry point against the workspace one (collected last on purpose).

Some hosts of the library cannot allocate device memory (a server plug-in that only gets its input and
output buffers, a process whose memory pool is fully reserved by another framework).  For them
``trj_argmax_accept_static`` keeps its scratch in a fixed array inside the library.  This test calls it
through the C ABI twice in a row on different inputs and checks every output against
``trj_argmax_accept`` and against the CPU oracle: integers bit-exact, margins to 1e-6 (the tolerance of the
other arg-max tests).
It must pass alone in a fresh process and after all other tests, because all calls share that one array.
"""
import numpy as np
import pytest
import torch

import oracle
import synth

pytestmark = pytest.mark.gpu


def make_case(trj, seed, rows_list, vocab, dtype):
    parents = [synth.random_tree(seed * 10 + i, m, min(5, max(1, m - 1)), 3) if m > 1 else np.array([-1], np.int32)
               for i, m in enumerate(rows_list)]
    depth = np.concatenate([trj.tree_from_parents(p)[0] for p in parents])
    logits = synth.logits(seed, sum(rows_list), vocab, dtype)
    off = np.concatenate([[0], np.cumsum(rows_list)]).astype(np.int32)
    best = logits.argmax(1)                                  # only used to plant drafts that get accepted
    tokens = np.concatenate([synth.planted_tokens(seed, p, best[off[i]:off[i + 1]], vocab, name=f"p{i}")
                             for i, p in enumerate(parents)])
    dev = lambda a, t: torch.from_numpy(np.ascontiguousarray(a)).to("cuda", t)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    host = {"logits": logits, "tokens": tokens, "parents": parents, "off": off}
    return (dev(logits, tdt), dev(tokens, torch.int32), dev(np.concatenate(parents), torch.int32),
            dev(depth, torch.int32), dev(off, torch.int32), host)


def fresh_outputs(trj, rows, batch):
    i32 = dict(dtype=torch.int32, device="cuda")
    return {"node_argmax": torch.full((rows,), -7, **i32), "margin": torch.full((rows,), -1.0, device="cuda"),
            "k_acc": torch.full((batch,), -7, **i32), "path": torch.full((batch, trj.PATH_STRIDE), -7, **i32),
            "bonus": torch.full((batch,), -7, **i32)}


def test_static_scratch_entry_point_matches_workspace_entry_point(trj):
    # two calls in a row on different shapes and dtypes: the second must not see the first one's leftovers
    for seed, rows_list, vocab, dtype in ((1, [64], 32000, "bf16"), (2, [5, 33, 1, 128, 17], 4099, "f32")):
        logits, tokens, parent, depth, off, host = make_case(trj, seed, rows_list, vocab, dtype)
        want = trj.argmax_accept(logits, tokens, parent, depth, off)
        got = fresh_outputs(trj, sum(rows_list), len(rows_list))
        trj.argmax_accept_static(logits, tokens, parent, depth, off, got)
        torch.cuda.synchronize()
        for name in ("node_argmax", "k_acc", "path", "bonus"):
            assert torch.equal(got[name], want[name]), name
        assert torch.allclose(got["margin"], want["margin"], rtol=0, atol=1e-6)
        assert int(want["k_acc"].max()) >= 1                 # the planted drafts make the walk non-trivial
        # ... and against the definition itself
        pred = oracle.node_argmax(host["logits"])
        np.testing.assert_array_equal(got["node_argmax"].cpu().numpy(), pred)
        np.testing.assert_allclose(got["margin"].cpu().numpy(), oracle.top2_margin(host["logits"]), rtol=0, atol=1e-6)
        o = host["off"]
        for b, par in enumerate(host["parents"]):
            k, path, bonus = oracle.accept_path(host["tokens"][o[b]:o[b + 1]], par, pred[o[b]:o[b + 1]])
            assert int(got["k_acc"][b]) == k and int(got["bonus"][b]) == bonus
            assert got["path"][b, :k + 1].tolist() == path and (got["path"][b, k + 1:] == -1).all()


def test_static_scratch_entry_point_refuses_oversized_batches(trj):
    rows = trj.STATIC_MAX_ROWS + 1
    logits = torch.zeros(rows, 8, device="cuda")
    z = torch.zeros(rows, dtype=torch.int32, device="cuda")
    off = torch.tensor([0, rows], dtype=torch.int32, device="cuda")
    with pytest.raises(trj.TrjError) as e:
        trj.argmax_accept_static(logits, z, z, z, off, fresh_outputs(trj, rows, 1))
    assert e.value.status == 2 and "built-in scratch" in str(e.value)
    # the total does not lift the per-tree limit: one tree of MAX_ROWS + 1 rows is refused before any launch
    rows = trj.MAX_ROWS + 1
    z = torch.zeros(rows, dtype=torch.int32, device="cuda")
    off = torch.tensor([0, rows], dtype=torch.int32, device="cuda")
    with pytest.raises(trj.TrjError) as e:
        trj.argmax_accept_static(torch.zeros(rows, 8, device="cuda"), z, z, z, off, fresh_outputs(trj, rows, 1))
    assert e.value.status == 2 and "at most" in str(e.value)
