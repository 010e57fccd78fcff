/*
 * trj.h -- C ABI of the TR-Jacobi verification step on one B200 (sm_100a).
 *
 * One verification step of tree-based retrieval-augmented Jacobi decoding
 * (paper Section 3.3): a token tree that merges the Jacobi window with
 * retrieved draft branches is scored by ONE model forward against the KV cache
 * (token-tree verification, Section 2.2 / Appendix B), the greedy longest
 * accepted root-to-leaf path is chosen (Section 3.3, Eq. 1) and the K/V of the
 * accepted rows is kept contiguous in the cache.
 *
 * Conventions that hold for every entry point
 * -------------------------------------------
 * Pointers   "dev" pointers are CUDA device addresses of the current device,
 *            "host" pointers are ordinary host addresses.  The caller allocates
 *            and owns every buffer; the library borrows it for the duration of
 *            the call (weights and workspace: for the lifetime of the context)
 *            and frees nothing it did not allocate.  The library allocates no
 *            DEVICE memory: all device scratch comes from caller-provided
 *            workspaces (one exception: trj_argmax_accept_static keeps its
 *            scratch in a fixed array of the library's device image).  A model
 *            context owns a few host-side objects of its own: small pinned
 *            staging buffers, a stream, an event and the CUDA graphs of its
 *            step; trj_destroy releases them.
 * Streams    `stream` is a cudaStream_t passed as void* (NULL = default
 *            stream).  Device entry points only enqueue work; results are in
 *            device memory once the stream has been synchronised.  Entry
 *            points whose name ends in _host copy to and from host buffers and
 *            synchronise the stream before returning.
 * Errors     Every function returns a trj_status.  Shapes, capacities and
 *            pointers are checked on the host before anything is launched, so
 *            an invalid call launches nothing.  Nothing aborts, throws or
 *            prints.  trj_last_error gives a message for the calling thread's
 *            most recent failure.  Every device-side wait of the tensor-core
 *            kernels is bounded; one that expires leaves TRJ_ETIMEOUT in a
 *            status word (of the op's workspace, or of the model context) and
 *            the kernel returns normally.  trj_step_host returns that status
 *            itself; after the asynchronous model calls ask trj_device_status.
 *            A shape that the tensor-core kernels are written for is never
 *            run on a slower kernel because a workspace is short or misaligned:
 *            that is TRJ_ECAPACITY / TRJ_EINVAL.
 * Layouts    All tensors are dense, row-major, innermost dimension last.
 *            dtype is TRJ_BF16 (bf16 storage, fp32 accumulation) or TRJ_F32.
 *            KV cache: [L][B][Hkv][max_seq][D] (Hkv = K/V heads: H, or fewer with
 *            grouped-query attention); sequence b has seq_len[b]
 *            committed rows; during a step the M_b tree rows of sequence b
 *            live at cache rows seq_len[b] .. seq_len[b] + M_b - 1.
 * Trees      A tree is a parent-pointer array in topological order:
 *            parent[0] = -1 (row 0 is the root = the last committed token,
 *            whose K/V is not cached yet) and 0 <= parent[i] < i.  depth[i] is
 *            the number of edges from the root.  anc is the ancestor-or-self
 *            bitmask: bit (j % 64) of word anc[i * anc_words + j / 64] is set
 *            iff row j is row i or one of its ancestors.  A batch of trees is
 *            ragged: rows of sequence b are row_off[b] .. row_off[b+1] - 1 and
 *            parent / anc bit indices are local to the sequence.
 * Limits     At most TRJ_MAX_ROWS rows per tree, TRJ_MAX_BATCH sequences.
 */
#ifndef TRJ_H
#define TRJ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TRJ_MAX_ROWS  128      /* tree rows per sequence, root included          */
#define TRJ_MAX_BATCH 64       /* sequences per call                             */
#define TRJ_PATH_STRIDE 128    /* int32 slots per sequence in `path` arrays      */
#define TRJ_MAX_TOPK  10       /* candidates per row that a top-K call can return */

typedef enum {
    TRJ_OK = 0,
    TRJ_EINVAL = 1,        /* bad pointer, shape, tree or enum                   */
    TRJ_ECAPACITY = 2,     /* rows, batch, sequence length or workspace too small */
    TRJ_ECUDA = 3,         /* a CUDA runtime call failed                          */
    TRJ_ETIMEOUT = 4,      /* a bounded device-side wait expired                  */
    TRJ_EUNSUPPORTED = 5   /* valid request that this build has no kernel for     */
} trj_status;

typedef enum { TRJ_F32 = 0, TRJ_BF16 = 1 } trj_dtype;

typedef struct trj_ctx trj_ctx;    /* opaque model context */

/* LLaMA-family decoder shape: pre-norm, RMSNorm, rotary embedding (half-split
 * pairing, base rope_theta), multi-head or grouped-query attention, SwiGLU,
 * untied LM head.  The paper's main models (Table 2) are of the LLaMA-3 family:
 * grouped-query attention (n_kv_heads = 8 for 32 query heads) and a 128 256-way
 * vocabulary. */
typedef struct {
    int32_t n_layers, d_model, n_heads, head_dim, d_ff, vocab;
    float   rms_eps, rope_theta;
    int32_t dtype;                 /* trj_dtype of weights, activations and cache */
    int32_t max_batch, max_seq, max_rows;   /* capacities the workspace is sized for */
    int32_t n_kv_heads;            /* K/V heads; 0 = n_heads; must divide n_heads: query head h
                                      reads K/V head h / (n_heads / n_kv_heads)              */
} trj_model_cfg;

/* Device pointers to the weights, borrowed for the lifetime of the context.
 * Every matrix is [d_out][d_in].  The per-layer members are HOST arrays of
 * n_layers device pointers.  wqkv stacks Wq (H*D rows), Wk, Wv (Hkv*D rows each); w_gate_up stacks the
 * SwiGLU gate rows over the up rows.  Norm gains are fp32 vectors [d_model]. */
typedef struct {
    const void*  embed;            /* [vocab][d_model]  dtype                     */
    const void*  lm_head;          /* [vocab][d_model]  dtype                     */
    const float* final_norm;       /* [d_model]                                   */
    const float* const* attn_norm; /* [L] -> [d_model]                            */
    const void*  const* wqkv;      /* [L] -> [(H+2*Hkv)*D][d_model]               */
    const void*  const* wo;        /* [L] -> [d_model][H*D]                       */
    const float* const* mlp_norm;  /* [L] -> [d_model]                            */
    const void*  const* w_gate_up; /* [L] -> [2*d_ff][d_model]                    */
    const void*  const* w_down;    /* [L] -> [d_model][d_ff]                      */
} trj_weights;

const char* trj_last_error(void);
/* Library version string; also a cheap "does it load" probe. */
const char* trj_version(void);

/* ------------------------------------------------------------------------
 * build_tree (host, integers only).  Section 3.3: every path of the tree is an
 * ordinary Jacobi trajectory and retrieved drafts get a path of their own;
 * Appendix B: the tree is verified through a sparse attention mask.
 *
 * Lays out row 0 = root, rows 1..W = the Jacobi window as a chain, then each of
 * the R retrieved branches (branch r = branches[r*branch_len .. +branch_len))
 * as a chain hanging off the root.  Writes tokens/parent/depth [M] and
 * anc [M * anc_words] (anc_words >= ceil(M/64)), M = 1 + W + R*branch_len, and
 * *n_rows = M.  All pointers host.  TRJ_ECAPACITY if M > max_rows or
 * max_rows > TRJ_MAX_ROWS; TRJ_EINVAL on NULL or negative sizes. */
trj_status trj_build_tree(int32_t root, const int32_t* window, int32_t W,
                          const int32_t* branches, int32_t R, int32_t branch_len,
                          int32_t max_rows, int32_t anc_words,
                          int32_t* tokens, int32_t* parent, int32_t* depth,
                          uint64_t* anc, int32_t* n_rows);

/* Same derivation for an arbitrary tree given by parent pointers (host):
 * validates parent (TRJ_EINVAL if parent[0] != -1 or parent[i] is not an
 * earlier row; TRJ_ECAPACITY if M > TRJ_MAX_ROWS or anc_words < ceil(M/64))
 * and writes depth [M] and anc [M * anc_words]. */
trj_status trj_tree_from_parents(const int32_t* parent, int32_t M, int32_t anc_words,
                                 int32_t* depth, uint64_t* anc);

/* Prompt-lookup retrieval (Section 3.3, host).  Key = last 2 tokens of
 * context[0..n) (which ends with the root), then the last 1; scanning
 * backwards, the branch_len tokens after each of the R most recent earlier
 * occurrences become a branch; a slot retrieval cannot fill holds ahead noise
 * (Eq. 4) context[draws[r*branch_len + j] % n].  Writes branches [R*branch_len]. */
trj_status trj_retrieve(const int32_t* context, int32_t n, int32_t R, int32_t branch_len,
                        const int64_t* draws, int32_t* branches);

/* Next Jacobi window (Section 3.3, host): the predictions below the winning row
 * `best` along its branch (lowest-index child at every level), then ahead noise
 * context[draws[i] % n] for the remaining slots i < W.  Writes window [W]. */
trj_status trj_refill_window(const int32_t* parent, const int32_t* node_argmax, int32_t M,
                             int32_t best, int32_t W, const int32_t* context, int32_t n,
                             const int64_t* draws, int32_t* window);

/* ------------------------------------------------------------------------
 * Tree-masked attention (Section 2.2, Appendix B), batched and ragged.
 *
 *   out[r][h] = sum_j softmax_j( q[r][h] . K[b][h][j] / sqrt(D) ) V[b][h][j]
 *
 * for row r of sequence b (local index i = r - row_off[b]), j ranging over the
 * cache rows 0 .. seq_len[b]-1 and those tree rows seq_len[b] + t whose bit t is
 * set in anc[r].
 *   q, out     dev [rows_total][H][D]   dtype
 *   k_cache,
 *   v_cache    dev [B][H][max_seq][D]   dtype (tree rows already stored in place)
 *   seq_len    dev [B] int32;  row_off dev [B+1] int32;  anc dev [rows_total][anc_words]
 *   max_rows   upper bound of rows per sequence (<= TRJ_MAX_ROWS)
 *   max_len    upper bound of seq_len[b] + rows of b, <= max_seq (sizes the KV split)
 *   workspace  dev, at least trj_tree_attention_workspace(...) bytes, 256-byte aligned;
 *              holds split-KV partial results, contents undefined afterwards.  Its first
 *              int32 is a status word: the kernels set it to TRJ_ETIMEOUT if a bounded
 *              device-side wait expires and never clear it (zero it to be able to read it).
 * TRJ_EUNSUPPORTED for a head_dim the build has no kernel for (supported: 64, 128). */
size_t trj_tree_attention_workspace(int32_t rows_total, int32_t B, int32_t H, int32_t D, int32_t max_len);
trj_status trj_tree_attention(const void* q, const void* k_cache, const void* v_cache,
                              const int32_t* seq_len, const int32_t* row_off, const uint64_t* anc,
                              int32_t anc_words, int32_t B, int32_t rows_total, int32_t max_rows,
                              int32_t H, int32_t D, int32_t max_seq, int32_t max_len, int32_t dtype,
                              void* out, void* workspace, size_t workspace_bytes, void* stream);
/* The same with grouped-query attention (LLaMA-3 family, Table 2): H query heads over Hkv K/V heads, H a
 * multiple of Hkv; k_cache / v_cache are [B][Hkv][max_seq][D] and query head h reads K/V head h / (H / Hkv).
 * Hkv == H is trj_tree_attention. */
trj_status trj_tree_attention_gqa(const void* q, const void* k_cache, const void* v_cache,
                                  const int32_t* seq_len, const int32_t* row_off, const uint64_t* anc,
                                  int32_t anc_words, int32_t B, int32_t rows_total, int32_t max_rows,
                                  int32_t H, int32_t Hkv, int32_t D, int32_t max_seq, int32_t max_len, int32_t dtype,
                                  void* out, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * Per-node arg-max fused with greedy longest-path acceptance (Eq. 1; Section
 * 3.3: candidate generation and verification share the forward, so every row's
 * prediction is an output).
 *
 *   node_argmax[r] = argmax_v logits[r][v]           (ties -> smallest v)
 *   ok[0] = 1;  ok[i] = ok[parent[i]] && tokens[i] == node_argmax[parent[i]]
 *   best  = accepted row of largest depth (ties -> smallest row);  k = depth[best]
 *   path  = rows root..best (k+1 entries, local indices, rest -1);  bonus = node_argmax[best]
 *
 *   logits     dev [rows_total][V] dtype;  tokens/parent/depth dev [rows_total] int32
 *   node_argmax dev [rows_total];  margin dev [rows_total] fp32 or NULL (top-1 minus top-2 logit)
 *   k_acc, bonus dev [B];  path dev [B][TRJ_PATH_STRIDE]
 *   workspace  dev, >= trj_argmax_accept_workspace(rows_total, B) bytes, 256-byte aligned.
 *              The library keeps tickets in it that must be zero on entry of the
 *              FIRST call; every call leaves them zero again.
 * Inputs must be finite. */
size_t trj_argmax_accept_workspace(int32_t rows_total, int32_t B);
trj_status trj_argmax_accept(const void* logits, int32_t dtype, int32_t V,
                             const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                             const int32_t* row_off, int32_t B, int32_t rows_total,
                             int32_t* node_argmax, float* margin,
                             int32_t* k_acc, int32_t* path, int32_t* bonus,
                             void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * Top-K siblings (Appendix B: the tree template holds, as siblings, the K most
 * likely tokens of a draft position; the candidates of the first draft position
 * carry most of what the tree adds).
 *
 * trj_topk_accept is trj_argmax_accept that also returns, for every row, the ids
 * of its K largest logits, best first (larger logit first, equal logits by
 * ascending id), in topk [rows_total][K] (dev int32; column 0 equals
 * node_argmax).  1 <= K <= TRJ_MAX_TOPK.  Acceptance is unchanged: a row is
 * accepted iff its token is the arg-max of its parent.  workspace: dev, >=
 * trj_topk_accept_workspace() bytes, 256-byte aligned, zero before the first
 * call; every call leaves it zero again.
 *
 * trj_node_topk: the same top-K of the logits that the latest trj_verify_step on
 * ctx produced (rows_total as in that call); launches only.
 *
 * trj_refill_tree (host): draft tokens of the next step for a static template
 * with top-K siblings.  The template is parent [M] plus rank [M]: rank[i] = r >=
 * 0 makes row i the r-th best candidate of its position (siblings under one
 * parent carry ranks 0, 1, 2, ...), rank[i] = -1 - j makes it slot j of the
 * retrieval path and it takes retrieved[j].  Candidates for depth d come from the
 * d-th row below the winner `best` along its own path (lowest-index child at
 * every level): row i of depth d and rank r takes topk[that row][r]; depths the
 * path does not reach are ahead noise context[draws[i-1] % n] (Eq. 4).  Writes
 * tokens [M-1] (rows 1..M-1; the root is the step's bonus token).  With a chain
 * and ranks 0 this is trj_refill_window.  All pointers host. */
size_t trj_topk_accept_workspace(void);
trj_status trj_topk_accept(const void* logits, int32_t dtype, int32_t V, int32_t K,
                           const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                           const int32_t* row_off, int32_t B, int32_t rows_total,
                           int32_t* topk, int32_t* node_argmax, float* margin,
                           int32_t* k_acc, int32_t* path, int32_t* bonus,
                           void* workspace, size_t workspace_bytes, void* stream);
trj_status trj_node_topk(trj_ctx* ctx, int32_t rows_total, int32_t K, int32_t* topk, void* stream);
trj_status trj_refill_tree(const int32_t* parent, const int32_t* rank, int32_t M, const int32_t* topk, int32_t K,
                           int32_t best, const int32_t* context, int32_t n, const int64_t* draws,
                           const int32_t* retrieved, int32_t n_retrieved, int32_t* tokens);

/* ------------------------------------------------------------------------
 * trj_argmax_accept for callers that cannot hand over a workspace (the paper has
 * no counterpart; this is a deployment convenience).  Some hosts of this library
 * are not allowed to allocate device memory at all: a plug-in of an inference
 * server that is given nothing but its input and output buffers, or a process
 * whose memory pool was reserved in full at start-up by another framework, so
 * that a cudaMalloc from inside a call would fail or break that framework's
 * accounting.  For them the scratch (tickets and per-slice arg-max candidates)
 * lives in a fixed array inside the library's device image, TRJ_STATIC_MAX_ROWS
 * rows' worth (about 96 KB), which every GPU that loads the library keeps for the
 * lifetime of the process.  Same inputs, outputs and results as
 * trj_argmax_accept.  The call allocates nothing, neither device nor pinned
 * memory.
 *   - rows_total > TRJ_STATIC_MAX_ROWS is refused with TRJ_ECAPACITY (use the
 *     workspace variant for larger batches).  The total does not lift the
 *     per-tree limit: a tree still holds at most TRJ_MAX_ROWS rows, and
 *     rows_total > B * TRJ_MAX_ROWS is refused with TRJ_ECAPACITY as well.
 *   - The first call on a device looks up the array's device address (a one-time
 *     set-up done with that device current); make that first call outside any
 *     stream capture (inside one it is refused with TRJ_EINVAL).
 *   - All calls on a device share the one array.  The tickets are cleared at the
 *     start of every call, so the previous call's contents do not matter, but two
 *     calls whose kernels overlap on the GPU (for instance on different
 *     streams) corrupt each other: serialise them. */
#define TRJ_STATIC_MAX_ROWS 1024
trj_status trj_argmax_accept_static(const void* logits, int32_t dtype, int32_t V,
                                    const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                    const int32_t* row_off, int32_t B, int32_t rows_total,
                                    int32_t* node_argmax, float* margin,
                                    int32_t* k_acc, int32_t* path, int32_t* bonus, void* stream);

/* ------------------------------------------------------------------------
 * KV compaction of the accepted path (implied by Section 3.3: decoding
 * continues from the accepted tokens).  For every layer, head and both K and
 * V, row seq_len[b] + path[b][j] moves to row seq_len[b] + j, j = 1..k_acc[b]
 * (row 0, the root, is already in place); then seq_len[b] += k_acc[b] + 1.
 * Bit-exact copy; source and destination ranges may overlap.
 *   k_cache, v_cache  dev [L][B][H][max_seq][D] dtype, modified in place (H = heads of the cache: the
 *                     K/V heads of a grouped-query model)
 *   seq_len dev [B] (updated);  k_acc dev [B];  path dev [B][TRJ_PATH_STRIDE] */
trj_status trj_compact_rows(void* k_cache, void* v_cache, int32_t L, int32_t B, int32_t H,
                            int32_t max_seq, int32_t D, int32_t dtype, int32_t* seq_len,
                            const int32_t* k_acc, const int32_t* path, void* stream);

/* ------------------------------------------------------------------------
 * Model context: the whole verification step of a LLaMA-shaped decoder.
 * workspace: dev, >= trj_workspace_bytes(cfg), 256-byte aligned, zero-filled by
 * the caller before trj_create, owned by the caller, used by every call on ctx.
 * The cache passed to the calls below is [n_layers][max_batch][Hkv][max_seq][D]. */
size_t     trj_workspace_bytes(const trj_model_cfg* cfg);
trj_status trj_create(const trj_model_cfg* cfg, const trj_weights* weights,
                      void* workspace, size_t workspace_bytes, trj_ctx** out);
trj_status trj_destroy(trj_ctx* ctx);

/* verify_step (Section 3.3): ONE forward of the decoder over all tree rows.
 * Embeds tokens, runs every layer (RMSNorm, QKV projection, rotary embedding at
 * position seq_len[b] + depth, K/V of the tree rows written to cache rows
 * seq_len[b] + i, tree-masked attention, output projection, SwiGLU MLP), the
 * final norm and the LM head, and writes node_argmax [rows_total] (Eq. 1),
 * margin [rows_total] when not NULL and, when logits is not NULL, the fp32
 * logits [rows_total][vocab].  seq_len is not changed.  All pointers dev.
 * B <= cfg.max_batch, rows per sequence <= cfg.max_rows and seq_len[b] + rows
 * <= max_len <= cfg.max_seq must hold (the caller's contract for device-held
 * lengths; max_len is the host-known bound used for launch sizing). */
trj_status trj_verify_step(trj_ctx* ctx, void* k_cache, void* v_cache, const int32_t* seq_len,
                           const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                           const uint64_t* anc, int32_t anc_words, const int32_t* row_off,
                           int32_t B, int32_t rows_total, int32_t max_rows, int32_t max_len,
                           int32_t* node_argmax, float* margin, float* logits, void* stream);

/* The same verification step (Section 3.3) for a decoder whose weights are
 * split over several devices (the 70B models of Table 2 do not fit one): a rank's
 * context is created from a cfg with n_heads / R query heads, n_kv_heads / R K/V
 * heads and d_ff / R feed-forward columns, d_model and vocab whole, and from the
 * matching slices of the weights: the rows of wqkv of its heads (its query
 * heads, then its key heads, then its value heads), the columns of wo of its
 * heads, its gate rows then its up rows of w_gate_up, its columns of w_down;
 * embedding, norms and LM head whole.  Its cache holds its K/V heads only.
 *
 * The decoder is 2 * n_layers + 1 segments (trj_tp_segments): 2 l is the
 * attention half of layer l, 2 l + 1 its feed-forward half, the last one the
 * final norm and the LM head.  Every segment but the last leaves, in the
 * exchange buffer (trj_tp_exchange_buffer: dev fp32 [rows_total][d_model], part
 * of the workspace), this rank's partial sum of the half's output projection.
 * The caller adds the buffers of all ranks, in place and to the same bits on
 * every rank (an all-reduce on `stream`), before it runs the next segment, which
 * adds the sum to the residual stream.  Order of calls: trj_tp_begin (checks as
 * trj_verify_step, embeds the tokens), trj_tp_segment for 0, 1, 2, ... in this
 * order (anything else: TRJ_EINVAL), trj_tp_finish (arg-max, margin and logits
 * as trj_verify_step; every rank computes the same).  The pointers given to
 * trj_tp_begin must stay valid until trj_tp_finish.  With R = 1 the sequence
 * computes what trj_verify_step computes, up to the order of a few fp32
 * additions (a half's split-K pieces are summed before they join the residual
 * stream instead of one by one).  Launches only; all pointers
 * dev except trj_tp_exchange_buffer's two results (host). */
int32_t    trj_tp_segments(const trj_ctx* ctx);
trj_status trj_tp_begin(trj_ctx* ctx, void* k_cache, void* v_cache, const int32_t* seq_len,
                        const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                        const uint64_t* anc, int32_t anc_words, const int32_t* row_off,
                        int32_t B, int32_t rows_total, int32_t max_rows, int32_t max_len, void* stream);
trj_status trj_tp_segment(trj_ctx* ctx, int32_t segment, void* stream);
trj_status trj_tp_exchange_buffer(const trj_ctx* ctx, float** partial, size_t* count);
trj_status trj_tp_finish(trj_ctx* ctx, int32_t* node_argmax, float* margin, float* logits, void* stream);

/* accept (Section 3.3): longest accepted path from node_argmax; see
 * trj_argmax_accept for the rule and the output layout.  All pointers dev. */
trj_status trj_accept(trj_ctx* ctx, const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                      const int32_t* row_off, int32_t B, int32_t rows_total, const int32_t* node_argmax,
                      int32_t* k_acc, int32_t* path, int32_t* bonus, void* stream);

/* compact_kv: trj_compact_rows over all layers of the context's cache shape. */
trj_status trj_compact_kv(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t B,
                          const int32_t* k_acc, const int32_t* path, void* stream);

/* Prefill of sequence b: scores n prompt tokens (dev int32) as chain trees of at
 * most cfg.max_rows rows (a chain tree is causal attention), appends their K/V
 * at seq_len[b] and advances seq_len[b] by n; *first_token (dev) receives the
 * greedy prediction after the last prompt token (Eq. 1). */
trj_status trj_prefill(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t b,
                       const int32_t* tokens, int32_t n, int32_t* first_token, void* stream);

/* One whole decode step from HOST buffers for batch 1 (the call a decoding loop
 * makes): builds the tree from root/window/branches (trj_build_tree), copies it
 * to the device, runs verify_step + accept + compact_kv, copies the result back
 * and synchronises `stream`.
 *   host in : root, window [W], branches [R*branch_len]
 *   host out: tokens/parent [M] (the tree that was scored), node_argmax [M],
 *             *k_acc, path [TRJ_PATH_STRIDE], *bonus, *n_rows
 *   dev     : k_cache, v_cache, seq_len [1] (advanced by k_acc + 1)
 *   max_len : host-known bound of seq_len[0] + M
 * From the second call on a context the launch sequence is captured once per
 * (tree rows, launch geometry, buffer addresses) into a CUDA graph (on a stream of
 * the context) and that graph is launched on `stream`; it runs after everything
 * already enqueued there and has completed when the call returns. */
trj_status trj_step_host(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t max_len,
                         int32_t root, const int32_t* window, int32_t W,
                         const int32_t* branches, int32_t R, int32_t branch_len,
                         int32_t* tokens, int32_t* parent, int32_t* n_rows, int32_t* node_argmax,
                         int32_t* k_acc, int32_t* path, int32_t* bonus, void* stream);

/* ------------------------------------------------------------------------
 * Drafting and refill on the device: the integer work between two verification
 * steps, so that a decode loop needs no host round trip per step.  Same rules
 * as trj_retrieve / trj_build_tree / trj_refill_window (Section 3.3: drafts are
 * retrieved from the tokens seen so far and the window is refilled from the
 * chosen path's own predictions; Eq. 4: ahead noise), on device buffers.
 * All pointers dev; launches only, nothing is synchronised.
 *
 * trj_draft_tokens: tokens [1 + W + R*branch_len] of the next tree in the fixed
 * layout of trj_build_tree: root = context[n_ctx - 1], then window [W], then R
 * retrieved branches.  draws [W + R*branch_len] int64 >= 0; slots [W, ...) feed
 * the branches' ahead noise (context[draw % n_ctx]).  R <= 64.
 *
 * trj_commit_refill: appends tokens[path[1..k]] and *bonus to context
 * (capacity ints; *n_ctx += k + 1), then writes the next window [W]:
 * node_argmax of the lowest-index child, level by level, below path[k], then
 * ahead noise context[draws[i] % n_ctx] on the grown context.  A context that
 * would overflow is left untouched and *overflow (may be null) is set to 1. */
trj_status trj_draft_tokens(const int32_t* context, const int32_t* n_ctx, const int32_t* window, int32_t W,
                            int32_t R, int32_t branch_len, const int64_t* draws, int32_t* tokens, void* stream);
trj_status trj_commit_refill(const int32_t* tokens, const int32_t* parent, const int32_t* node_argmax, int32_t M,
                             const int32_t* k_acc, const int32_t* path, const int32_t* bonus, int32_t* context,
                             int32_t capacity, int32_t* n_ctx, int32_t W, const int64_t* draws, int32_t* window,
                             int32_t* overflow, void* stream);

/* n_steps whole decode steps for batch 1 with everything resident on the device
 * (Section 3.3: draft, verify, accept, commit, refill): per step trj_draft_tokens, the verification forward, arg-max +
 * acceptance, KV compaction and trj_commit_refill are enqueued on `stream`; the
 * host is not involved between steps and the call does not wait for them.
 *   dev in/out: k_cache, v_cache, seq_len [1]; context [capacity] with *n_ctx
 *               valid tokens (prompt + generated; the last one is the next root,
 *               so seq_len[0] == *n_ctx - 1); window [W] (the next window)
 *   dev in    : draws [n_steps][W + R*branch_len] int64 >= 0 (step i uses row i:
 *               slots [W, ...) for its retrieval, slots [0, W) for its refill)
 *   dev out   : k_log [n_steps] accepted draft tokens per step (may be null)
 *   host      : n_ctx_now = the value of *n_ctx at the time of the call (used for
 *               the capacity checks: every step commits at most
 *               max(W, branch_len) + 1 tokens)
 * TRJ_ECAPACITY if the context buffer, cfg.max_seq or cfg.max_rows cannot take
 * the worst case; nothing is enqueued then. */
trj_status trj_decode_device(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t* context,
                             int32_t capacity, int32_t* n_ctx, int32_t n_ctx_now, int32_t* window, int32_t W,
                             int32_t R, int32_t branch_len, const int64_t* draws, int32_t n_steps,
                             int32_t* k_log, void* stream);

/* The same loop over a static tree template with top-K siblings (Appendix B;
 * template = parent [M] + rank [M] as for trj_refill_tree, HOST arrays; the rows
 * of rank -1-j are one retrieval path of n_retrieved slots).  Per step, all on
 * the device: the tree's tokens (root = the last committed token, the drafts
 * the previous refill left, the retrieval path refreshed from the current
 * context: slot j takes the j-th token after the most recent earlier occurrence
 * of the context's last two tokens, then of its last token, else ahead noise),
 * the verification forward, per-row top-K (K <= TRJ_MAX_TOPK) + acceptance, KV
 * compaction, then commit and the refill rule of trj_refill_tree.
 *   dev in/out: k_cache, v_cache, seq_len [1], context [capacity], *n_ctx as for
 *               trj_decode_device; drafts [M - 1]: the draft tokens of rows
 *               1 .. M-1 for the first step on entry (retrieval rows are
 *               ignored), those for the next step on return
 *   dev in    : draws [n_steps][M - 1 + n_retrieved] int64 >= 0: step i uses
 *               row i, slots [0, M - 1) for its refill, the rest for the ahead
 *               noise of its retrieval path
 *   dev out   : k_log [n_steps] (may be null)
 *   host      : parent, rank, n_ctx_now (every step commits at most the
 *               template's depth + 1 tokens)
 * Errors as trj_decode_device; a rank >= K or a retrieval slot >= n_retrieved
 * is TRJ_EINVAL. */
trj_status trj_decode_device_tree(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t* context,
                                  int32_t capacity, int32_t* n_ctx, int32_t n_ctx_now, const int32_t* parent,
                                  const int32_t* rank, int32_t M, int32_t K, int32_t n_retrieved, int32_t* drafts,
                                  const int64_t* draws, int32_t n_steps, int32_t* k_log, void* stream);

/* An external source of drafts for trj_decode_device and trj_decode_device_tree (there it feeds the start of the
 * retrieval path instead of branch 0) (Section 3.3: retrieved drafts get a path of their own; where
 * they are retrieved from is open).  stream [n] (dev int32) holds the source's guess for the token at context
 * position i in stream[i]; in step s of a later trj_decode_device call the first take[s] (dev int32 [n_steps],
 * clipped to branch_len and to n) tokens of retrieved branch 0 come from stream, starting at the position after
 * the root, instead of from prompt lookup.  Borrowed until replaced; stream == NULL removes the source.  With
 * guesses of a known quality this sets how many drafts a step accepts: the benchmark uses it to run the loop at
 * the acceptance lengths the paper reports instead of the zero of random drafts on random weights. */
trj_status trj_set_draft_source(trj_ctx* ctx, const int32_t* stream, int32_t n, const int32_t* take, int32_t n_steps);

/* ------------------------------------------------------------------------
 * The projections as a stand-alone op: y[M][N] (fp32) = x[M][K] . w[N][K]^T,
 * x and w of `dtype`, all dev.  Used by the model path for every projection
 * and exposed for measurement.  workspace: dev, >= trj_gemm_workspace(M, N, K)
 * bytes, 256-byte aligned (split-K partial sums); its first int32 is a status
 * word with the same meaning as in trj_tree_attention. */
size_t     trj_gemm_workspace(int32_t M, int32_t N, int32_t K);
trj_status trj_gemm(const void* x, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                    int32_t dtype, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------
 * Device-side time-outs (no counterpart in the paper).
 * trj_device_status: synchronises `stream` and reads the context's two status
 * words (projections, attention).  TRJ_OK if no bounded device-side wait has
 * expired since the words were last cleared, TRJ_ETIMEOUT otherwise; with
 * clear != 0 the words are then reset.  After a time-out the results of the
 * affected step are undefined and the context's workspace should be zero-filled
 * again before it is reused (tickets and partial sums may be half-written).
 * trj_selftest_wait_expiry: launches one CTA in which one thread waits, with a
 * limit of `polls` polls (1 .. 2^21), on a barrier that nobody arrives at, using
 * the same wait routine as the tensor-core kernels.  The wait gives up, writes
 * TRJ_ETIMEOUT to *status (dev int32) and the kernel returns by itself: a way to
 * see the error path work without anything going wrong. */
trj_status trj_device_status(trj_ctx* ctx, int32_t clear, void* stream);
trj_status trj_selftest_wait_expiry(int32_t* status, int32_t polls, void* stream);

/* Index checks (no counterpart in the paper).  The kernels that index the cache with device-held lengths and
 * paths (rotary + K/V append, attention, compaction) never touch a row outside the cache: an access that a
 * length or path breaking the caller's contract (seq_len[b] + rows <= max_len <= max_seq, path entries inside the
 * tree) would push outside is skipped, lengths are brought inside the cache before they size a loop, and nothing
 * traps; the result of such a step is unspecified.  A library built with -DTRJ_DEBUG also records which check
 * fired: trj_debug_flags synchronises the device, writes the bits seen since the last call to *flags (host) and
 * clears them: 1 a K/V append past the cache, 2 a compaction source or destination past the cache or a negative
 * path entry, 4 seq_len + rows beyond the cache in the generic attention kernel.  The default build records
 * nothing and returns TRJ_EUNSUPPORTED. */
trj_status trj_debug_flags(int32_t* flags);

/* ------------------------------------------------------------------------
 * Measurement aids (no counterpart in the paper).
 * trj_launch_count: kernel launches this process has enqueued through the
 * library so far (every launch is counted on the host when it is enqueued).
 * trj_profile_enable(ctx, 1): from now on every kernel launch made on behalf of
 * ctx is bracketed by two CUDA events on its stream (cost: two event records
 * per launch; at most 8192 launches are kept between reads).
 * trj_profile_read: waits for the recorded events, sums the device time and
 * the launches per category (0 element-wise/norm, 1 projections, 2 rotary +
 * K/V append, 3 tree attention, 4 arg-max/accept, 5 compaction) into
 * ms[TRJ_PROF_CATEGORIES] / launches[TRJ_PROF_CATEGORIES] (host) and clears
 * the record unless keep != 0.  Launches made while the stream is being captured
 * record their events as nodes of the graph, so every replay of that graph times
 * itself again (read with keep = 1 after each replay). */
#define TRJ_PROF_CATEGORIES 6
uint64_t   trj_launch_count(void);
/* Clock stamps of the per-layer kernels.  Only a library built with -DTRJ_TIMELINE records them (the default
 * build returns TRJ_EUNSUPPORTED from both calls and carries no instrumentation).  Every launch of a kind below
 * records the time (ns, GPU global timer) at which its first CTA got past the wait for the previous kernel and the
 * time at which its last CTA ended.  trj_timeline_reset clears the record (enqueued on `stream`);
 * trj_timeline_read copies the launches of one kind since the last reset, in launch order, to begin_ns / end_ns
 * (host, max_launches each) and their number to *n_launches; synchronise the device first. */
#define TRJ_TL_RMSNORM   0   /* residual add + RMSNorm        */
#define TRJ_TL_GEMM      1   /* projection                     */
#define TRJ_TL_ROPE      2   /* rotary embedding + K/V append  */
#define TRJ_TL_ATTENTION 3   /* tree attention                 */
#define TRJ_TL_SWIGLU    4   /* SwiGLU                         */
#define TRJ_TL_EMBED     5   /* embedding gather               */
#define TRJ_TL_KINDS     6
trj_status trj_timeline_reset(void* stream);
/* Most CTAs of the projection kernel that were ever resident on one SM at the same time since the library was loaded
 * (clock-stamp build only; synchronise the device first): shows that two CTAs really share an SM, which the occupancy
 * calculator denies for a kernel that allocates tensor memory. */
trj_status trj_timeline_ctas_per_sm(int32_t* peak);
trj_status trj_timeline_read(int32_t kind, int32_t max_launches, uint64_t* begin_ns, uint64_t* end_ns, int32_t* n_launches);
/* Programmatic dependent launch (on by default): the kernels of a step are launched so that each may
 * be scheduled, and may prefetch weights, while its predecessor in the stream is still running.
 * trj_set_pdl(0) launches them fully serialised instead (for comparison).  Process-wide; set it
 * before the first step of a context, because a cached CUDA graph keeps the mode it was captured in. */
void       trj_set_pdl(int32_t on);
trj_status trj_profile_enable(trj_ctx* ctx, int32_t on);
trj_status trj_profile_read(trj_ctx* ctx, float* ms, int32_t* launches, int32_t keep);

#ifdef __cplusplus
}
#endif
#endif /* TRJ_H */
