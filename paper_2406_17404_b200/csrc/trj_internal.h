// Internal declarations shared by the translation units of libtrj (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "trj.h"

namespace trj {

// ---- error plumbing (thread-local message, never throws) -------------------
trj_status fail(trj_status code, const char* fmt, ...);
#define TRJ_CHECK_CUDA(expr)                                                        \
    do {                                                                            \
        cudaError_t e__ = (expr);                                                   \
        if (e__ != cudaSuccess)                                                     \
            return ::trj::fail(TRJ_ECUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
    } while (0)
#define TRJ_REQUIRE(cond, code, ...)                         \
    do {                                                     \
        if (!(cond)) return ::trj::fail(code, __VA_ARGS__);  \
    } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline size_t dtype_size(int32_t dt) { return dt == TRJ_BF16 ? 2 : 4; }

// ---- host-side tree helpers (host_tree.cpp) ---------------------------------
trj_status tree_from_parents_impl(const int32_t* parent, int32_t M, int32_t anc_words,
                                  int32_t* depth, uint64_t* anc);

// ---- programmatic dependent launch -----------------------------------------------------------------
// Inside a chain (a ChainScope on the calling thread: the model forward and the steps that follow it),
// kernels are launched so that a kernel may be scheduled while its predecessor in the stream is still
// running: every such kernel first lets ITS successor start (launch_dependents) and then waits for its
// predecessor to finish and flush (wait) before it touches any data the predecessor may write.
// The first kernel of a forward (the embedding) is the chain's fence: it waits BEFORE it lets its
// successor start.  A chain kernel that has started therefore knows that everything enqueued before that
// embedding is complete, so ahead of its own wait it may read what only earlier work wrote: the batch
// geometry (seq_len, row_off, depth), weights, and cache rows below seq_len.  Anything written inside the
// chain is read after the wait.  Outside a chain (the op-level entry points, whose predecessor is
// unknown) kernels are launched without the attribute, and both instructions do nothing.
bool pdl_enabled();
void set_pdl(bool on);
bool chain_active();                      // this thread is inside a ChainScope and PDL is enabled
struct ChainScope { ChainScope(); ~ChainScope(); ChainScope(const ChainScope&) = delete; };
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_prologue() { pdl_launch_dependents(); pdl_wait(); }

template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(bool programmatic, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                             Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// A kernel of a chain (see above): programmatic only inside a ChainScope.
template <typename... KArgs, typename... Args>
cudaError_t launch_chain(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    return launch_dependent(chain_active(), kernel, grid, block, smem, st, static_cast<Args&&>(args)...);
}
#endif

// ---- optional clock stamps (builds with -DTRJ_TIMELINE): one table per translation unit that holds kernels
#ifdef TRJ_TIMELINE
cudaError_t timeline_reset_generic(cudaStream_t st);
cudaError_t timeline_reset_gemm(cudaStream_t st);
cudaError_t timeline_reset_attention(cudaStream_t st);
int timeline_read_generic(int kind, int max_launches, uint64_t* begin_ns, uint64_t* end_ns);
int timeline_read_gemm(int kind, int max_launches, uint64_t* begin_ns, uint64_t* end_ns);
int timeline_gemm_ctas_per_sm();          // most CTAs of the plain projection kernel ever resident on one SM
int timeline_read_attention(int kind, int max_launches, uint64_t* begin_ns, uint64_t* end_ns);
#endif

#ifdef TRJ_DEBUG
cudaError_t debug_flags_read(int* flags);      // synchronises the device, returns and clears the index-check flags
#endif

// ---- launch accounting: every kernel launch of the library passes through count_launch() -------
void count_launch();
uint64_t launches_so_far();

// ---- generic kernels (kernels_generic.cu); every launcher only enqueues ------
// Geometry of a ragged batch of trees over a KV cache slab of one layer.
struct Batch {
    const int32_t* seq_len;   // [B] dev
    const int32_t* row_off;   // [B+1] dev
    int32_t B, rows_total, max_rows, max_len;
    // 1: every cache row below seq_len was written before the chain of kernels this batch is launched in began, so a
    // kernel may fetch such rows ahead of its wait for its predecessor; 0: some were written inside the chain
    int32_t cached_rows_final = 1;
    // 1: every sequence of the batch reads and extends the cache of sequence 0 of the slab (the pieces of a prompt
    // chunk: piece j is a "sequence" whose cached rows are the prompt so far plus the pieces before it)
    int32_t shared_cache = 0;
};

// Weights of a LATER projection that a projection kernel may ask for ahead of time.  When the kernel before a
// projection leaves SMs free and HBM idle (the attention kernel of a decoding step does both), the projection's
// first `ctas` CTAs get those SMs at once and spend their wait requesting the first `bytes` of `w` ([N][K] bf16)
// into L2, so that the later projection starts from L2 instead of HBM; before that they request the first
// `self_bytes` of the projection's OWN weights the same way.  ctas = 0: nothing is requested.
struct WeightPrefetch { const void* w; int32_t N, K; size_t bytes; int32_t ctas; size_t self_bytes; };

// A projection result that may still be in split-K pieces: value(i) = sum over s < splits of ptr[s * stride + i].
struct Parts { const float* ptr; int32_t splits; size_t stride; };
inline Parts whole(const float* p) { return Parts{p, 1, 0}; }

// Arg-max fused into a projection's epilogue (Eq. 1 needs every row's arg-max, not the logits): every epilogue warp
// leaves, for every activation row, the best value, its output index (ties: the smaller index) and the runner-up value
// among its 32 outputs of the tile.  Table layout: entry ((row * tiles + tile) * 4 + warp); tiles = ceil(N / 128).
// Only for launches with one K range and one row block (gemm_top_table_ok); y is still written unless store_y == 0.
struct TopEntry { float v1; int32_t i1; float v2; };
struct TopTable { TopEntry* entries; int32_t store_y; };
bool gemm_top_table_ok(int32_t M, int32_t N, int32_t K, int32_t dtype, bool pair);
inline size_t gemm_top_table_entries(int32_t rows, int32_t N) { return (size_t)rows * ((N + 127) / 128) * 4; }

cudaError_t launch_embed(const void* embed, int32_t dtype, const int32_t* tokens, float* h,
                         int32_t rows, int32_t d, cudaStream_t st);
// h += add (when add != nullptr, h is updated in place); x = rmsnorm(h) * gain, stored as dtype.
// In bf16 models x is written as a bf16 pair: x (hi) and x_lo (the rounding error of hi); x_lo may be null.
cudaError_t launch_add_rmsnorm(float* h, const Parts& add, const float* gain, void* x, void* x_lo, int32_t dtype,
                               int32_t rows, int32_t d, float eps, cudaStream_t st);
// y[M][N] fp32 = (x + x_lo)[M][K] . w[N][K]^T (x_lo may be null), plain shared-memory tiled FMA kernel.
cudaError_t launch_gemm_simt(const void* x, const void* x_lo, const void* w, float* y, int32_t M, int32_t N,
                             int32_t K, int32_t dtype, cudaStream_t st);
// tcgen05 / TMA projection kernel (gemm_sm100.cu): bf16, K >= 64 and a multiple of 8 (rows of 16-byte multiples).  The workspace
// (gemm_tc_workspace bytes, 256-byte aligned) starts with a status word that a device-side wait sets to
// TRJ_ETIMEOUT if it expires; the rest holds split-K partial sums.
bool gemm_tc_supported(const void* x, const void* x_lo, const void* w, const float* y, int32_t M, int32_t N, int32_t K,
                       int32_t dtype);
size_t gemm_tc_workspace(int32_t M, int32_t N, int32_t K);
cudaError_t launch_gemm_tc(const void* x, const void* x_lo, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                           void* workspace, cudaStream_t st, Parts* parts, const WeightPrefetch* ahead = nullptr,
                           int* status = nullptr, const TopTable* top = nullptr);
// The tcgen05 kernel for every shape it is written for (bf16, K >= 64 and a multiple of 8, N a multiple of 4), the plain
// kernel for the rest (fp32 models, odd sizes).  A shape of the first kind whose workspace is too small or
// misaligned is an error (cudaErrorInvalidValue), never a silent detour through the plain kernel.  With `parts`
// non-null the split-K pieces are left unreduced in the workspace for the consumer to add (*parts says where);
// otherwise y holds the finished result.  `status` (may be null: the workspace's first word) receives
// TRJ_ETIMEOUT when a bounded device-side wait expires.
bool gemm_tc_shape(int32_t M, int32_t N, int32_t K, int32_t dtype);
cudaError_t launch_gemm(const void* x, const void* x_lo, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                        int32_t dtype, void* workspace, size_t workspace_bytes, cudaStream_t st, Parts* parts = nullptr,
                        const WeightPrefetch* ahead = nullptr, int* status = nullptr, const TopTable* top = nullptr);

// Rotary embedding of q and k at position seq_len[b] + depth[row]; q -> q_out [rows][H][D];
// k, v -> cache rows seq_len[b] + local row of the layer slab [B][Hkv][max_seq][D].  The projection result has
// (H + 2 * Hkv) * D values per row: H query heads, then Hkv key heads, then Hkv value heads.
cudaError_t launch_rope_kv_write(const Parts& qkv, const double* inv_freq, const int32_t* depth,
                                 const Batch& bt, void* q_out, void* k_slab, void* v_slab, int32_t dtype,
                                 int32_t H, int32_t Hkv, int32_t D, int32_t max_seq, cudaStream_t st);
// Attention: H query heads over Hkv K/V heads (query head h reads K/V head h / (H / Hkv)).
cudaError_t launch_tree_attention_generic(const void* q, const void* k_slab, const void* v_slab,
                                          const uint64_t* anc, int32_t anc_words, const Batch& bt,
                                          int32_t H, int32_t Hkv, int32_t D, int32_t max_seq, int32_t dtype,
                                          void* out, void* out_lo, cudaStream_t st);
// tcgen05 / TMA tree attention (attn_sm100.cu): bf16, head_dim 128.  Workspace: status word in the first
// 256 bytes, then split-KV partial results.
bool tree_attention_tc_supported(int32_t D, int32_t dtype, int32_t max_rows);
size_t tree_attention_tc_workspace(int32_t B, int32_t H);
int tree_attention_grid(int32_t B, int32_t H, int32_t max_len);     // CTAs the tcgen05 kernel is launched with
cudaError_t launch_tree_attention_tc(const void* q, const void* k_slab, const void* v_slab, const uint64_t* anc,
                                     int32_t anc_words, const Batch& bt, int32_t H, int32_t Hkv, int32_t max_seq, void* out,
                                     void* out_lo, void* workspace, cudaStream_t st, int* status = nullptr);
// The tcgen05 kernel for bf16 with head_dim 128, the generic kernel for the rest (fp32, head_dim 64).  A bf16 /
// head_dim-128 call whose workspace is too small or misaligned is an error (cudaErrorInvalidValue), never a
// silent detour.  out_lo (may be null) receives the rounding error of `out` as a second tensor of the same
// type, for the projection that follows.  `status`: as for launch_gemm.
cudaError_t launch_tree_attention(const void* q, const void* k_slab, const void* v_slab, const uint64_t* anc,
                                  int32_t anc_words, const Batch& bt, int32_t H, int32_t Hkv, int32_t D, int32_t max_seq,
                                  int32_t dtype, void* out, void* out_lo, void* workspace, size_t workspace_bytes,
                                  cudaStream_t st, int* status = nullptr);
// One CTA waits, with a poll limit, on a barrier nobody arrives at (self-test of the time-out path).
cudaError_t launch_wait_expiry_selftest(int* status, uint32_t polls, cudaStream_t st);

// Device-side drafting and refill (device_loop.cu); all pointers are device pointers.  `step` (may be null: step 0)
// is a device counter that selects the step's slice of `draws` ([steps][W + R * Lr]) and is advanced by the commit.
// An external source of drafts for the decode loop: stream[i] (i < n) is its guess for the token at context position
// i; take[s] is how many of them step s puts at the start of retrieved branch 0.  stream == nullptr: none.
struct DraftSource { const int32_t* stream; int32_t n; const int32_t* take; };
cudaError_t launch_draft_tokens(const int32_t* context, const int32_t* n_ctx, const int32_t* window, int32_t W, int32_t R,
                                int32_t Lr, const int64_t* draws, const int32_t* step, int32_t* tokens, cudaStream_t st,
                                const DraftSource& src = DraftSource{nullptr, 0, nullptr});
cudaError_t launch_commit_refill(const int32_t* tokens, const int32_t* parent, const int32_t* node_argmax, int32_t M,
                                 const int32_t* k_acc, const int32_t* path, const int32_t* bonus, int32_t* context,
                                 int32_t capacity, int32_t* n_ctx, int32_t W, int32_t draws_per_step, const int64_t* draws,
                                 int32_t* step, int32_t* window, int32_t* k_log, int32_t* overflow, cudaStream_t st);
// The same two steps for a static tree template with top-K siblings (parent / depth / rank [M] on the device): the
// tokens of a step (root, the drafts the previous refill left, the retrieval path refreshed from the context; the
// retrieved tokens are kept in retr), and the commit + refill of the drafts from the per-row top-K table.  draws of
// step s: draws[s][0 .. M-2] refill, draws[s][M-1 .. M-2+n_retr] retrieval.
cudaError_t launch_template_tokens(const int32_t* context, const int32_t* n_ctx, const int32_t* drafts, const int32_t* rank,
                                   int32_t M, int32_t n_retr, const int64_t* draws, const int32_t* step, int32_t* tokens,
                                   int32_t* retr, cudaStream_t st, const DraftSource& src = DraftSource{nullptr, 0, nullptr});
cudaError_t launch_commit_refill_tree(const int32_t* tokens, const int32_t* parent, const int32_t* depth, const int32_t* rank,
                                      const int32_t* topk, int32_t K, int32_t M, const int32_t* k_acc, const int32_t* path,
                                      const int32_t* bonus, int32_t* context, int32_t capacity, int32_t* n_ctx, int32_t n_retr,
                                      const int64_t* draws, int32_t* step, const int32_t* retr, int32_t* drafts, int32_t* k_log,
                                      int32_t* overflow, cudaStream_t st);

// act[M][f] (dtype) = silu(gu[:, :f]) * gu[:, f:]
cudaError_t launch_swiglu(const Parts& gu, void* act, void* act_lo, int32_t dtype, int32_t rows, int32_t f,
                          cudaStream_t st);

// Arg-max over the vocabulary and/or acceptance.  do_argmax: compute node_argmax (+margin) from
// logits; do_accept: walk the tree and write k_acc/path/bonus.  ws: tickets + partials.
size_t argmax_workspace_bytes(int32_t rows_total, int32_t B);
cudaError_t launch_argmax_accept(const void* logits, int32_t dtype, int32_t V,
                                 const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                 const int32_t* row_off, int32_t B, int32_t rows_total,
                                 int32_t* node_argmax, float* margin, int32_t* k_acc, int32_t* path,
                                 int32_t* bonus, bool do_argmax, bool do_accept, void* ws, cudaStream_t st);

// Per-row top-K (K = 1: arg-max; ids best first into topk [rows][K] when not null; node_argmax and margin as above)
// and, with do_accept, the acceptance walk.  One CTA per row; ws: one ticket per sequence (topk_workspace_bytes, zero
// before the first call, left zero by every call).
size_t topk_workspace_bytes();
cudaError_t launch_topk_accept(const void* logits, int32_t dtype, int32_t V, int32_t K,
                               const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                               const int32_t* row_off, int32_t B, int32_t rows_total, int32_t* topk,
                               int32_t* node_argmax, float* margin, int32_t* k_acc, int32_t* path,
                               int32_t* bonus, bool do_accept, void* ws, cudaStream_t st);

// Arg-max + acceptance from the table a projection's epilogue left (gemm_top_table_entries): entries_per_row
// candidates per row, merged with the full (value, index) order.
cudaError_t launch_argmax_table_accept(const TopEntry* table, int32_t entries_per_row, const int32_t* tokens,
                                       const int32_t* parent, const int32_t* depth, const int32_t* row_off, int32_t B,
                                       int32_t rows_total, int32_t* node_argmax, float* margin, int32_t* k_acc,
                                       int32_t* path, int32_t* bonus, bool do_accept, void* ws, cudaStream_t st);

// Same kernel with its scratch in a file-scope device array of the library (no workspace argument).
cudaError_t launch_argmax_accept_static(const void* logits, int32_t dtype, int32_t V,
                                        const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                        const int32_t* row_off, int32_t B, int32_t rows_total,
                                        int32_t* node_argmax, float* margin, int32_t* k_acc, int32_t* path,
                                        int32_t* bonus, cudaStream_t st);

// tickets (may be null): TRJ_MAX_BATCH zero-initialised counters; with them the lengths are advanced by the same
// kernel (the CTA that finishes a sequence last), without them by a second launch.
cudaError_t launch_compact(void* k_cache, void* v_cache, int32_t L, int32_t B_cache, int32_t B, int32_t H,
                           int32_t max_seq, int32_t D, int32_t dtype, int32_t* seq_len,
                           const int32_t* k_acc, const int32_t* path, cudaStream_t st, unsigned int* tickets = nullptr);
// row_off = {0, m} and seq_len[b] += delta: small bookkeeping used by prefill.
cudaError_t launch_set_chunk(int32_t* row_off2, int32_t m, cudaStream_t st);
// Geometry of a prefill chunk of m rows whose attention treats n_sub pieces of `sub` rows (the last one shorter) as
// the sequences of one batch: lens[j] = *seq_len_b + j * sub, off_all = {0, m}, off_pieces[j] = min(j * sub, m).
cudaError_t launch_prefill_geometry(const int32_t* seq_len_b, int32_t* lens, int32_t n_sub, int32_t sub, int32_t m,
                                    int32_t* off_all, int32_t* off_pieces, cudaStream_t st);
cudaError_t launch_bump_len(int32_t* seq_len_b, int32_t delta, cudaStream_t st);

}  // namespace trj
