"""CPU oracle for the TR-Jacobi verification step  --  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 numpy restatement of what one verification forward step of
tree-based retrieval-augmented Jacobi decoding computes (paper Section 3.3,
Section 2.2 for token-tree verification, Eq. 1 for the greedy target,
Appendix B for the tree template).  It exists so that the CUDA path has
something independent to be compared against; only the tests, the smoke check
and the CPU-baseline leg of the benchmark may import it.  It shares no code
with the CUDA path and never imports it.

What is written out here is the definition, not an optimised algorithm: one
dense matmul per projection, attention as an explicit softmax over the visible
set of every row, acceptance as a parent-pointer recurrence.  There is no
tiling, no online softmax and no fusion.

Precision: every floating-point step is fp64.  Inputs arrive as float32 arrays
whose values are already representable in the storage type of the config
(bf16 or fp32) and are widened exactly.  In a bf16 model the operands of the
attention op (q and the K/V cache rows) are bf16 tensors by the config's
definition, so the decoder rounds them to bf16 where they are stored; nothing
else is rounded (the attention result feeds the output projection unrounded).

Readings taken where the paper is silent (each one is a free choice that
cannot change which tokens a greedy decoder commits, unless noted):

* Model.  The paper names LLaMA-family 7-8B decoders but prints no
  architecture.  Used here: pre-norm decoder, RMSNorm (eps 1e-5), rotary
  embedding with the half-split pairing (i, i + D/2) and base 10000, multi-head
  attention scaled by 1/sqrt(D), SwiGLU MLP, no biases, untied LM head.  With
  grouped-query attention (LLaMA-3 family, Table 2) query head h reads K/V
  head h // (H / Hkv).
* Tree layout (Section 3.3, Appendix B).  The concrete 63-node template is a
  third-party artefact that the paper does not print; any parent-pointer tree
  with parent[i] < i is accepted.  ``build_tree`` lays out row 0 = root (the
  last committed token, whose K/V is not cached yet), rows 1..W = the Jacobi
  window as a chain, then every retrieved branch as its own chain hanging off
  the root, in retrieval order, without merging equal prefixes.
* Positions.  Row i sits at position S + depth[i]; siblings share a position.
* Mask (Section 2.2, Appendix B).  Row i sees the S cached rows and those tree
  rows that are its ancestors or itself.
* Acceptance (Section 3.3, "longest accept-length path").  Row i is accepted
  iff its parent is accepted and its token equals the arg-max at its parent.
  The deepest accepted row wins; among equally deep rows the smallest row
  index wins.  Arg-max ties go to the smallest token id.
* Step output.  With k = depth of the winning row, the step commits the k
  draft tokens on the path plus one bonus token (the arg-max at the winning
  row), i.e. at least one token per step, like an autoregressive step.
* Compaction (implied by continuing to decode).  K/V of path[j] moves to cache
  row S + j for j = 0..k; the new length is S + k + 1.
* Refill (Section 3.3).  New root = bonus.  New window = the arg-max at the
  rows below the winner along its own branch (lowest-index child at every
  level), then ahead noise up to W tokens.
* Top-K trees (Appendix B: most of the tree's benefit comes from the
  candidates of the first draft position; the 63-node template itself is
  third-party and not printed).  A template is ``parent`` plus a rank per row: siblings
  under one parent carry ranks 0, 1, 2, ... and hold the rank-th most likely
  token for their position; rows of negative rank form the retrieval path.
  The candidates for depth d come from the d-th row below the winner along
  its own path (lowest-index child at every level), so all rows of one depth
  and rank carry the same token; depths the path does not reach are ahead
  noise.  Top-K order: larger logit first, equal logits by ascending id.
  With a chain template this is the window refill above.
* Ahead noise (Eq. 4).  Uniform over all tokens committed so far; the raw
  random draws are inputs.
* Retrieval (Section 3.3, prompt lookup).  Key = the last g committed tokens
  (g = 2, falling back to g = 1); the context is scanned backwards and the
  Lr tokens following each of the R most recent earlier occurrences become a
  branch; missing tokens are ahead noise.

Pins (tests/test_oracle_*.py): chain tree == causal attention == token-by-token
autoregressive forward; greedy TR-Jacobi output == greedy autoregressive
output; brute-force enumeration of all root-to-node paths; subtree
independence and row-permutation invariance; softmax closed forms; rotary
relative-position invariant; an independent library decoder
(transformers' LLaMA) on the tiny config; hand-worked acceptance cases.
Not pinned by the paper ("parity unpinned"): the free choices listed above
(rotary pairing and base, eps, noise distribution, retrieval key length and
order, tree template) -- they are fixed by this file and matched by the CUDA
path, and the library-decoder pin fixes the model-side ones to the common
LLaMA convention.
"""
from .tree import (ancestor_mask, pack_mask, build_tree, depths, retrieve, ahead_noise,
                   refill_window, refill_tree, continuation_rows, validate_tree)
from .attention import tree_attention
from .accept import node_argmax, node_topk, accept_path, compact_rows, top2_margin
from .model import Decoder, KVCache, autoregressive_greedy, tr_jacobi_generate, tr_jacobi_generate_tree

__all__ = [
    "ancestor_mask", "pack_mask", "build_tree", "depths", "retrieve", "ahead_noise",
    "refill_window", "refill_tree", "continuation_rows", "validate_tree", "tree_attention", "node_argmax",
    "node_topk", "accept_path", "compact_rows", "top2_margin", "Decoder", "KVCache",
    "autoregressive_greedy", "tr_jacobi_generate", "tr_jacobi_generate_tree",
]
