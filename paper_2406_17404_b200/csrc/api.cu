// C ABI of libtrj: argument checks, workspace carving and the launch sequence of a verification step.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <utility>
#include <vector>
#include <cstdlib>
#include "trj_internal.h"

using namespace trj;

namespace {

bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }
bool dtype_ok(int32_t dt) { return dt == TRJ_F32 || dt == TRJ_BF16; }

// Carves consecutive 256-byte aligned regions out of a workspace.
struct Carver {
    char* base; size_t off = 0;
    explicit Carver(void* p) : base((char*)p) {}
    template <typename T> T* take(size_t count) {
        T* r = (T*)(base + off);
        off += align_up(sizeof(T) * count, 256);
        return r;
    }
};

}  // namespace

// ---------------------------------------------------------------------------- op-level entry points
extern "C" size_t trj_tree_attention_workspace(int32_t rows_total, int32_t B, int32_t H, int32_t D, int32_t max_len) {
    (void)rows_total; (void)max_len;
    return D == 128 ? tree_attention_tc_workspace(B, H) : 256;
}

extern "C" trj_status trj_tree_attention(const void* q, const void* k_cache, const void* v_cache,
                                         const int32_t* seq_len, const int32_t* row_off, const uint64_t* anc,
                                         int32_t anc_words, int32_t B, int32_t rows_total, int32_t max_rows,
                                         int32_t H, int32_t D, int32_t max_seq, int32_t max_len, int32_t dtype,
                                         void* out, void* workspace, size_t workspace_bytes, void* stream) {
    return trj_tree_attention_gqa(q, k_cache, v_cache, seq_len, row_off, anc, anc_words, B, rows_total, max_rows, H, H, D,
                                  max_seq, max_len, dtype, out, workspace, workspace_bytes, stream);
}

extern "C" trj_status trj_tree_attention_gqa(const void* q, const void* k_cache, const void* v_cache,
                                             const int32_t* seq_len, const int32_t* row_off, const uint64_t* anc,
                                             int32_t anc_words, int32_t B, int32_t rows_total, int32_t max_rows,
                                             int32_t H, int32_t Hkv, int32_t D, int32_t max_seq, int32_t max_len, int32_t dtype,
                                             void* out, void* workspace, size_t workspace_bytes, void* stream) {
    TRJ_REQUIRE(Hkv >= 1 && H >= Hkv && H % Hkv == 0, TRJ_EINVAL, "tree_attention: %d query heads over %d K/V heads", H, Hkv);
    TRJ_REQUIRE(q && k_cache && v_cache && seq_len && row_off && anc && out, TRJ_EINVAL, "tree_attention: null pointer");
    TRJ_REQUIRE(dtype_ok(dtype), TRJ_EINVAL, "tree_attention: unknown dtype %d", dtype);
    TRJ_REQUIRE(B >= 1 && H >= 1 && rows_total >= 0 && max_rows >= 1, TRJ_EINVAL, "tree_attention: bad sizes");
    TRJ_REQUIRE(B <= TRJ_MAX_BATCH, TRJ_ECAPACITY, "tree_attention: batch %d exceeds %d", B, TRJ_MAX_BATCH);
    TRJ_REQUIRE(max_rows <= TRJ_MAX_ROWS, TRJ_ECAPACITY, "tree_attention: %d rows per tree exceed %d", max_rows, TRJ_MAX_ROWS);
    TRJ_REQUIRE(anc_words >= (max_rows + 63) / 64, TRJ_EINVAL, "tree_attention: anc_words %d too small", anc_words);
    TRJ_REQUIRE(max_len <= max_seq, TRJ_ECAPACITY, "tree_attention: max_len %d exceeds cache rows %d", max_len, max_seq);
    TRJ_REQUIRE(D == 64 || D == 128, TRJ_EUNSUPPORTED, "tree_attention: head_dim %d (supported: 64, 128)", D);
    TRJ_REQUIRE(aligned(q, 16) && aligned(k_cache, 16) && aligned(v_cache, 16) && aligned(out, 16), TRJ_EINVAL,
                "tree_attention: tensors must be 16-byte aligned");
    TRJ_REQUIRE(workspace && workspace_bytes >= trj_tree_attention_workspace(rows_total, B, H, D, max_len),
                TRJ_ECAPACITY, "tree_attention: workspace too small");
    TRJ_REQUIRE(aligned(workspace, 256), TRJ_EINVAL, "tree_attention: workspace must be 256-byte aligned");
    if (rows_total == 0) return TRJ_OK;
    Batch bt{seq_len, row_off, B, rows_total, max_rows, max_len};
    TRJ_CHECK_CUDA(launch_tree_attention(q, k_cache, v_cache, anc, anc_words, bt, H, Hkv, D, max_seq, dtype, out, nullptr,
                                         workspace, workspace_bytes, (cudaStream_t)stream));
    return TRJ_OK;
}

extern "C" size_t trj_argmax_accept_workspace(int32_t rows_total, int32_t B) {
    return argmax_workspace_bytes(rows_total, B);
}

extern "C" trj_status trj_argmax_accept(const void* logits, int32_t dtype, int32_t V,
                                        const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                        const int32_t* row_off, int32_t B, int32_t rows_total,
                                        int32_t* node_argmax, float* margin,
                                        int32_t* k_acc, int32_t* path, int32_t* bonus,
                                        void* workspace, size_t workspace_bytes, void* stream) {
    TRJ_REQUIRE(logits && tokens && parent && depth && row_off && node_argmax && k_acc && path && bonus,
                TRJ_EINVAL, "argmax_accept: null pointer");
    TRJ_REQUIRE(dtype_ok(dtype), TRJ_EINVAL, "argmax_accept: unknown dtype %d", dtype);
    TRJ_REQUIRE(V >= 1 && B >= 1 && rows_total >= B, TRJ_EINVAL, "argmax_accept: bad sizes (every tree has a root)");
    TRJ_REQUIRE(B <= TRJ_MAX_BATCH, TRJ_ECAPACITY, "argmax_accept: batch %d exceeds %d", B, TRJ_MAX_BATCH);
    TRJ_REQUIRE(rows_total <= B * TRJ_MAX_ROWS, TRJ_ECAPACITY, "argmax_accept: too many rows");
    TRJ_REQUIRE(workspace && aligned(workspace, 256) && workspace_bytes >= argmax_workspace_bytes(rows_total, B),
                TRJ_ECAPACITY, "argmax_accept: workspace too small or misaligned");
    TRJ_CHECK_CUDA(launch_topk_accept(logits, dtype, V, 1, tokens, parent, depth, row_off, B, rows_total, nullptr, node_argmax,
                                      margin, k_acc, path, bonus, true, workspace, (cudaStream_t)stream));
    return TRJ_OK;
}

extern "C" size_t trj_topk_accept_workspace(void) { return topk_workspace_bytes(); }

extern "C" trj_status trj_topk_accept(const void* logits, int32_t dtype, int32_t V, int32_t K,
                                      const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                      const int32_t* row_off, int32_t B, int32_t rows_total,
                                      int32_t* topk, int32_t* node_argmax, float* margin,
                                      int32_t* k_acc, int32_t* path, int32_t* bonus,
                                      void* workspace, size_t workspace_bytes, void* stream) {
    TRJ_REQUIRE(logits && tokens && parent && depth && row_off && topk && node_argmax && k_acc && path && bonus,
                TRJ_EINVAL, "topk_accept: null pointer");
    TRJ_REQUIRE(dtype_ok(dtype), TRJ_EINVAL, "topk_accept: unknown dtype %d", dtype);
    TRJ_REQUIRE(K >= 1 && K <= TRJ_MAX_TOPK && K <= V, TRJ_EINVAL, "topk_accept: K = %d outside 1..min(%d, V)", K, TRJ_MAX_TOPK);
    TRJ_REQUIRE(V >= 1 && B >= 1 && rows_total >= B, TRJ_EINVAL, "topk_accept: bad sizes (every tree has a root)");
    TRJ_REQUIRE(B <= TRJ_MAX_BATCH, TRJ_ECAPACITY, "topk_accept: batch %d exceeds %d", B, TRJ_MAX_BATCH);
    TRJ_REQUIRE(rows_total <= B * TRJ_MAX_ROWS, TRJ_ECAPACITY, "topk_accept: too many rows");
    TRJ_REQUIRE(workspace && aligned(workspace, 256) && workspace_bytes >= topk_workspace_bytes(),
                TRJ_ECAPACITY, "topk_accept: workspace too small or misaligned");
    TRJ_CHECK_CUDA(launch_topk_accept(logits, dtype, V, K, tokens, parent, depth, row_off, B, rows_total, topk, node_argmax,
                                      margin, k_acc, path, bonus, true, workspace, (cudaStream_t)stream));
    return TRJ_OK;
}

extern "C" trj_status trj_argmax_accept_static(const void* logits, int32_t dtype, int32_t V,
                                               const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                               const int32_t* row_off, int32_t B, int32_t rows_total,
                                               int32_t* node_argmax, float* margin,
                                               int32_t* k_acc, int32_t* path, int32_t* bonus, void* stream) {
    TRJ_REQUIRE(logits && tokens && parent && depth && row_off && node_argmax && k_acc && path && bonus,
                TRJ_EINVAL, "argmax_accept_static: null pointer");
    TRJ_REQUIRE(dtype_ok(dtype), TRJ_EINVAL, "argmax_accept_static: unknown dtype %d", dtype);
    TRJ_REQUIRE(V >= 1 && B >= 1 && rows_total >= B, TRJ_EINVAL, "argmax_accept_static: bad sizes (every tree has a root)");
    TRJ_REQUIRE(B <= TRJ_MAX_BATCH, TRJ_ECAPACITY, "argmax_accept_static: batch %d exceeds %d", B, TRJ_MAX_BATCH);
    TRJ_REQUIRE(rows_total <= TRJ_STATIC_MAX_ROWS, TRJ_ECAPACITY,
                "argmax_accept_static: %d rows exceed the built-in scratch of %d rows; use trj_argmax_accept with a workspace",
                rows_total, TRJ_STATIC_MAX_ROWS);
    TRJ_REQUIRE(rows_total <= B * TRJ_MAX_ROWS, TRJ_ECAPACITY,
                "argmax_accept_static: %d rows in %d trees: a tree holds at most %d rows", rows_total, B, TRJ_MAX_ROWS);
    const cudaError_t e = launch_argmax_accept_static(logits, dtype, V, tokens, parent, depth, row_off, B, rows_total,
                                                      node_argmax, margin, k_acc, path, bonus, (cudaStream_t)stream);
    TRJ_REQUIRE(e != cudaErrorStreamCaptureUnsupported, TRJ_EINVAL,
                "argmax_accept_static: the first call on a device must be made outside stream capture");
    TRJ_CHECK_CUDA(e);
    return TRJ_OK;
}

extern "C" trj_status trj_compact_rows(void* k_cache, void* v_cache, int32_t L, int32_t B, int32_t H,
                                       int32_t max_seq, int32_t D, int32_t dtype, int32_t* seq_len,
                                       const int32_t* k_acc, const int32_t* path, void* stream) {
    TRJ_REQUIRE(k_cache && v_cache && seq_len && k_acc && path, TRJ_EINVAL, "compact_rows: null pointer");
    TRJ_REQUIRE(dtype_ok(dtype), TRJ_EINVAL, "compact_rows: unknown dtype %d", dtype);
    TRJ_REQUIRE(L >= 1 && B >= 1 && H >= 1 && max_seq >= 1 && D >= 1, TRJ_EINVAL, "compact_rows: bad sizes");
    TRJ_REQUIRE(B <= TRJ_MAX_BATCH, TRJ_ECAPACITY, "compact_rows: batch %d exceeds %d", B, TRJ_MAX_BATCH);
    TRJ_REQUIRE((D * dtype_size(dtype)) % 16 == 0 && aligned(k_cache, 16) && aligned(v_cache, 16), TRJ_EINVAL,
                "compact_rows: cache rows must be multiples of 16 bytes and 16-byte aligned");
    TRJ_CHECK_CUDA(launch_compact(k_cache, v_cache, L, B, B, H, max_seq, D, dtype, seq_len, k_acc, path,
                                  (cudaStream_t)stream));
    return TRJ_OK;
}

extern "C" size_t trj_gemm_workspace(int32_t M, int32_t N, int32_t K) {
    return gemm_tc_workspace(M, N, K);
}

extern "C" trj_status trj_gemm(const void* x, const void* w, float* y, int32_t M, int32_t N, int32_t K,
                               int32_t dtype, void* workspace, size_t workspace_bytes, void* stream) {
    TRJ_REQUIRE(x && w && y, TRJ_EINVAL, "gemm: null pointer");
    TRJ_REQUIRE(dtype_ok(dtype), TRJ_EINVAL, "gemm: unknown dtype %d", dtype);
    TRJ_REQUIRE(M >= 1 && N >= 1 && K >= 1, TRJ_EINVAL, "gemm: bad sizes");
    TRJ_REQUIRE(workspace && workspace_bytes >= trj_gemm_workspace(M, N, K), TRJ_ECAPACITY, "gemm: workspace too small");
    TRJ_REQUIRE(aligned(workspace, 256) && aligned(x, 16) && aligned(w, 16) && aligned(y, 16), TRJ_EINVAL,
                "gemm: workspace must be 256-byte aligned, tensors 16-byte aligned");
    TRJ_CHECK_CUDA(launch_gemm(x, nullptr, w, y, M, N, K, dtype, workspace, workspace_bytes, (cudaStream_t)stream));
    return TRJ_OK;
}

// ---------------------------------------------------------------------------- model context
struct trj_ctx {
    trj_model_cfg cfg;
    const void* embed; const void* lm_head; const float* final_norm;
    std::vector<const float*> attn_norm, mlp_norm;
    std::vector<const void*> wqkv, wo, w_gate_up, w_down;
    // workspace regions (device)
    float* h; float* y; float* logits;
    void* x; void* x_lo; void* q; void* act; void* act_lo;   // *_lo: low halves of split bf16 activations
    double* inv_freq;
    int sm_count;          // SMs of the device the context lives on
    void* argmax_ws; void* attn_ws; size_t attn_ws_bytes; void* gemm_ws; size_t gemm_ws_bytes;
    // chain-tree tables for prefill and the staging area of trj_step_host (device)
    int32_t* chain_depth; uint64_t* chain_anc; int32_t* chunk_row_off; int32_t* unit_row_off; int32_t* prefill_geo;
    unsigned int* compact_tickets;   // device: one counter per sequence for the compaction kernel
    int32_t* loop_state;   // device: [0] step counter, [1] context-overflow flag of trj_decode_device
    TopEntry* top_table; int32_t top_table_rows;   // arg-max candidates left by the LM head's epilogue, and how many rows it may hold
    int32_t lm_table_rows = 0;   // rows whose candidates the latest forward left there (0: it wrote logits only)
    int32_t* loop_tree;    // device: rank [TRJ_MAX_ROWS] | retrieved tokens [TRJ_MAX_ROWS] | top-K table [TRJ_MAX_ROWS][TRJ_MAX_TOPK]
    int32_t* step_in;      // tokens | parent | depth | row_off(2) | pad -> anc
    int32_t* step_out;     // node_argmax | k_acc | bonus | path | device status words (projections, attention)
    int32_t* dev_status;   // the two status words at the end of step_out: TRJ_ETIMEOUT once a bounded wait expired
    int32_t* pin_in; int32_t* pin_out;   // pinned host mirrors
    // optional per-launch device timing (trj_profile_enable)
    bool prof_on = false; std::vector<cudaEvent_t> prof_ev; std::vector<int> prof_cat; size_t prof_used = 0;
    // CUDA graphs of trj_step_host, one per (tree rows, attention grid, buffers)
    struct GraphEntry { int32_t M; int grid; void* k; void* v; void* len; cudaGraphExec_t exec; };
    std::vector<GraphEntry> graphs;
    // CUDA graphs of one step of trj_decode_device, keyed by every pointer and size the step depends on
    struct LoopGraph { std::vector<uint64_t> key; cudaGraphExec_t exec; };
    std::vector<LoopGraph> loop_graphs;
    cudaStream_t cap_stream = nullptr; cudaEvent_t order_ev = nullptr; uint64_t steps_done = 0;
    DraftSource draft_src{nullptr, 0, nullptr}; int32_t draft_src_steps = 0;   // trj_set_draft_source
    int32_t last_rows = 0, last_B = 0; const int32_t* last_row_off = nullptr;  // geometry of the latest trj_verify_step
    // the step a tensor-parallel rank is walking through segment by segment (trj_tp_begin .. trj_tp_finish)
    struct TpStep {
        bool open = false; int32_t next = 0; void* k_cache = nullptr; void* v_cache = nullptr;
        Batch bt{}; const int32_t* tokens = nullptr; const int32_t* parent = nullptr; const int32_t* depth = nullptr;
        const uint64_t* anc = nullptr; int32_t anc_words = 0;
    } tp;
};

namespace {

// Prefill scores a prompt in chunks of this many rows (the projections see them all at once, so the weights are
// streamed once per chunk); attention takes a chunk as a batch of pieces of at most TRJ_MAX_ROWS rows, at most 16 of
// them.  1024 rows: the projections of a 2048-token prompt take 52 ms against 56 ms with 512-row chunks; with 2048
// rows they take 47.5 ms but the 16-piece attention launches give the gain back.
constexpr int PREFILL_CHUNK = 1024;
constexpr int PREFILL_MAX_SUB = 16;
struct SubChunks { int n, sub; const int32_t* lens; const int32_t* off_pieces; };

constexpr int STEP_IN_INTS = 3 * TRJ_MAX_ROWS + 4;                       // + anc (2 words per row) after it
constexpr int STEP_IN_BYTES = STEP_IN_INTS * 4 + TRJ_MAX_ROWS * 2 * 8;
constexpr int STEP_STATUS_AT = TRJ_MAX_ROWS + 2 + TRJ_PATH_STRIDE;
constexpr int STEP_OUT_INTS = STEP_STATUS_AT + 2;

int kv_heads(const trj_model_cfg& c) { return c.n_kv_heads > 0 ? c.n_kv_heads : c.n_heads; }

size_t carve(const trj_model_cfg& c, void* ws, trj_ctx* ctx) {
    const size_t es = dtype_size(c.dtype);
    const int step_rows = c.max_batch * c.max_rows;          // rows of a verification step
    const int rows = std::max(step_rows, PREFILL_CHUNK);     // ... or of a prefill chunk
    const int HD = c.n_heads * c.head_dim;
    const int QKV = HD + 2 * kv_heads(c) * c.head_dim;
    const size_t wide = (size_t)std::max(std::max(QKV, 2 * c.d_ff), c.d_model);
    Carver cv(ws);
    float* h = cv.take<float>((size_t)rows * c.d_model);
    float* y = cv.take<float>((size_t)rows * wide);
    float* logits = cv.take<float>((size_t)step_rows * c.vocab);
    char* x = cv.take<char>((size_t)rows * std::max(c.d_model, HD) * es);
    char* x_lo = cv.take<char>((size_t)rows * std::max(c.d_model, HD) * es);
    char* q = cv.take<char>((size_t)rows * HD * es);
    char* act = cv.take<char>((size_t)rows * c.d_ff * es);
    char* act_lo = cv.take<char>((size_t)rows * c.d_ff * es);
    double* inv_freq = cv.take<double>(c.head_dim / 2);
    char* argmax_ws = cv.take<char>(argmax_workspace_bytes(step_rows, c.max_batch));
    // a prefill chunk's pieces are the sequences of one attention launch
    const size_t attn_bytes = trj_tree_attention_workspace(rows, std::max(c.max_batch, PREFILL_MAX_SUB), c.n_heads, c.head_dim, c.max_seq);
    char* attn_ws = cv.take<char>(attn_bytes);
    // every row count a call may bring (the K split, hence the space for partial sums, is not monotone in it)
    size_t gemm_bytes = 256;
    for (auto nk : {std::pair<int, int>{QKV, c.d_model}, {c.d_model, HD}, {2 * c.d_ff, c.d_model},
                    {c.d_model, c.d_ff}, {c.vocab, c.d_model}})
        for (int m = 1; m <= rows; ++m)
            gemm_bytes = std::max(gemm_bytes, gemm_tc_workspace(m, nk.first, nk.second));
    char* gemm_ws = cv.take<char>(gemm_bytes);
    int32_t* chain_depth = cv.take<int32_t>(PREFILL_CHUNK);
    int32_t* prefill_geo = cv.take<int32_t>(2 * PREFILL_MAX_SUB + 4);   // piece lengths, {0, m}, piece row offsets
    uint64_t* chain_anc = cv.take<uint64_t>((size_t)PREFILL_CHUNK * 2);   // row i: the chain mask of row i % (rows of a piece)
    int32_t* chunk_row_off = cv.take<int32_t>(2);
    int32_t* unit_row_off = cv.take<int32_t>(2);
    int32_t* step_in = (int32_t*)cv.take<char>(STEP_IN_BYTES);
    int32_t* step_out = cv.take<int32_t>(STEP_OUT_INTS);
    int32_t* loop_state = cv.take<int32_t>(64);
    int32_t* loop_tree = cv.take<int32_t>((size_t)TRJ_MAX_ROWS * (2 + TRJ_MAX_TOPK));
    const int top_rows = std::min(step_rows, 128);
    TopEntry* top_table = cv.take<TopEntry>(gemm_top_table_entries(top_rows, c.vocab));
    unsigned int* compact_tickets = cv.take<unsigned int>(TRJ_MAX_BATCH);
    if (ctx) {
        ctx->h = h; ctx->y = y; ctx->logits = logits; ctx->x = x; ctx->q = q; ctx->act = act;
        ctx->x_lo = c.dtype == TRJ_BF16 ? x_lo : nullptr; ctx->act_lo = c.dtype == TRJ_BF16 ? act_lo : nullptr;
        ctx->inv_freq = inv_freq; ctx->argmax_ws = argmax_ws; ctx->attn_ws = attn_ws; ctx->attn_ws_bytes = attn_bytes;
        ctx->gemm_ws = gemm_ws; ctx->gemm_ws_bytes = gemm_bytes;
        ctx->chain_depth = chain_depth; ctx->chain_anc = chain_anc; ctx->prefill_geo = prefill_geo;
        ctx->chunk_row_off = chunk_row_off; ctx->unit_row_off = unit_row_off;
        ctx->step_in = step_in; ctx->step_out = step_out; ctx->loop_state = loop_state; ctx->loop_tree = loop_tree; ctx->top_table = top_table; ctx->top_table_rows = top_rows;
        ctx->dev_status = step_out + STEP_STATUS_AT;
        ctx->compact_tickets = compact_tickets;
    }
    return cv.off;
}

trj_status check_cfg(const trj_model_cfg* c) {
    TRJ_REQUIRE(c, TRJ_EINVAL, "cfg: null");
    TRJ_REQUIRE(dtype_ok(c->dtype), TRJ_EINVAL, "cfg: unknown dtype %d", c->dtype);
    TRJ_REQUIRE(c->n_layers >= 1 && c->d_model >= 1 && c->n_heads >= 1 && c->d_ff >= 1 && c->vocab >= 1,
                TRJ_EINVAL, "cfg: non-positive dimension");
    TRJ_REQUIRE(c->head_dim == 64 || c->head_dim == 128, TRJ_EUNSUPPORTED, "cfg: head_dim %d (supported: 64, 128)", c->head_dim);
    TRJ_REQUIRE(c->n_kv_heads >= 0 && c->n_kv_heads <= c->n_heads && (c->n_kv_heads == 0 || c->n_heads % c->n_kv_heads == 0),
                TRJ_EINVAL, "cfg: %d K/V heads do not divide %d query heads", c->n_kv_heads, c->n_heads);
    TRJ_REQUIRE(c->max_batch >= 1 && c->max_batch <= TRJ_MAX_BATCH, TRJ_ECAPACITY, "cfg: max_batch %d outside 1..%d", c->max_batch, TRJ_MAX_BATCH);
    TRJ_REQUIRE(c->max_rows >= 1 && c->max_rows <= TRJ_MAX_ROWS, TRJ_ECAPACITY, "cfg: max_rows %d outside 1..%d", c->max_rows, TRJ_MAX_ROWS);
    TRJ_REQUIRE(c->max_seq >= c->max_rows, TRJ_EINVAL, "cfg: max_seq smaller than a tree");
    TRJ_REQUIRE(c->rms_eps >= 0.f && c->rope_theta > 0.f, TRJ_EINVAL, "cfg: bad eps or rope base");
    return TRJ_OK;
}

enum { PROF_ELEMENTWISE = 0, PROF_GEMM = 1, PROF_ROPE = 2, PROF_ATTENTION = 3, PROF_ARGMAX = 4, PROF_COMPACT = 5 };
constexpr size_t PROF_MAX_LAUNCHES = 8192;

// Inside a stream capture the records become event nodes of the graph (external events), so a replayed
// graph times its own kernels without any host gap in between.
unsigned prof_flags(cudaStream_t st) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) return cudaEventRecordDefault;
    return cs == cudaStreamCaptureStatusActive ? cudaEventRecordExternal : cudaEventRecordDefault;
}
void prof_begin(trj_ctx* ctx, int cat, cudaStream_t st) {
    if (!ctx->prof_on || ctx->prof_used >= PROF_MAX_LAUNCHES) return;
    ctx->prof_cat[ctx->prof_used] = cat;
    cudaEventRecordWithFlags(ctx->prof_ev[2 * ctx->prof_used], st, prof_flags(st));
}
void prof_end(trj_ctx* ctx, cudaStream_t st) {
    if (!ctx->prof_on || ctx->prof_used >= PROF_MAX_LAUNCHES) return;
    cudaEventRecordWithFlags(ctx->prof_ev[2 * ctx->prof_used + 1], st, prof_flags(st));
    ++ctx->prof_used;
}
#define LAUNCH(cat, expr)                  \
    do {                                   \
        prof_begin(ctx, cat, st);          \
        cudaError_t le__ = (expr);         \
        prof_end(ctx, st);                 \
        if (le__ != cudaSuccess) return fail(TRJ_ECUDA, "%s: %s", #expr, cudaGetErrorString(le__)); \
    } while (0)

#define LAUNCH_ON(stream_, cat, expr)      \
    do {                                   \
        prof_begin(ctx, cat, stream_);     \
        cudaError_t le__ = (expr);         \
        prof_end(ctx, stream_);            \
        if (le__ != cudaSuccess) return fail(TRJ_ECUDA, "%s: %s", #expr, cudaGetErrorString(le__)); \
    } while (0)

// What one forward works on.  lm_first/lm_rows select which rows reach the LM head (prefill only needs its last
// row).  b0 = first sequence of the cache the batch maps to.  `pieces` (prefill only): attention runs piece by
// piece, every piece a chain below all rows before it.
struct StepArgs {
    void* k_cache; void* v_cache; int32_t b0; Batch bt;
    const int32_t* tokens; const int32_t* depth; const uint64_t* anc; int32_t anc_words;
    int32_t lm_first, lm_rows; const SubChunks* pieces;
    int32_t lm_mode;   // 0: logits; 1: logits and the arg-max candidates of the epilogue; 2: the candidates only
};

// The decoder as 2 L + 1 segments: 2 l is the attention half of layer l (norm, QKV, rotary + cache write, tree
// attention, output projection), 2 l + 1 its feed-forward half (norm, gate/up, SwiGLU, down projection), 2 L the
// final norm and the LM head.  Every half ends in a projection whose result the next segment adds to the residual
// stream; `pr` carries it from segment to segment, in split-K pieces unless `finish_last` asks for the last
// segment's result as finished sums in ctx->y (what a tensor-parallel rank hands to the sum over ranks).
trj_status run_segments(trj_ctx* ctx, const StepArgs& a, int s0, int s1, Parts& pr, bool finish_last, cudaStream_t st) {
    const trj_model_cfg& c = ctx->cfg;
    const Batch& bt = a.bt;
    const int M = bt.rows_total, d = c.d_model, HD = c.n_heads * c.head_dim, Hkv = kv_heads(c);
    const int QKV = HD + 2 * Hkv * c.head_dim;
    const size_t es = dtype_size(c.dtype);
    const size_t seq_stride = (size_t)Hkv * c.max_seq * c.head_dim * es;           // one sequence of one layer
    // CTAs of the attention launch: what it leaves of the device is free while it runs (the plain kernel fills it)
    const bool attn_tc = ctx->attn_ws && ((uintptr_t)ctx->attn_ws % 256) == 0 &&
                         ctx->attn_ws_bytes >= tree_attention_tc_workspace(bt.B, c.n_heads) &&
                         tree_attention_tc_supported(c.head_dim, c.dtype, bt.max_rows);
    const int attn_grid = attn_tc ? tree_attention_grid(bt.B, c.n_heads, bt.max_len) : ctx->sm_count;
    int* const gemm_status = ctx->dev_status, *const attn_status = ctx->dev_status + 1;
    // measured on the 7B shape: 32-48 MB of the gate/up weights are worth 0.1 ms per step (16 MB: half of that, 64 MB:
    // a quarter); 12-20 MB of the output projection's own weights on top another 0.012 ms, more of them cost again
    constexpr size_t AHEAD_BYTES = (size_t)32 << 20, AHEAD_SELF_BYTES = (size_t)16 << 20;
    const SubChunks* pieces = a.pieces;
    for (int s = s0; s < s1; ++s) {
        const int l = s >> 1;
        Parts* const out_parts = (finish_last && s == s1 - 1) ? nullptr : &pr;
        if (s == 2 * c.n_layers) {
            LAUNCH(PROF_ELEMENTWISE, launch_add_rmsnorm(ctx->h, pr, ctx->final_norm, ctx->x, ctx->x_lo, c.dtype, M, d,
                                                        c.rms_eps, st));
            if (a.lm_rows > 0) {
                const size_t off = (size_t)a.lm_first * d * es;
                // a verification step keeps every row's logits in place; prefill wants one row and gets it in row 0
                float* lm_out = pieces ? ctx->logits : ctx->logits + (size_t)a.lm_first * c.vocab;
                // Eq. 1 needs every row's arg-max, not its logits: when the caller says so and the launch keeps all of
                // a row's partial sums in one accumulator, the epilogue leaves one candidate per 32 outputs and the
                // logits are written only if they are wanted as well
                const bool table = a.lm_mode != 0 && !pieces && a.lm_first == 0 && a.lm_rows == M && M <= ctx->top_table_rows &&
                                   gemm_top_table_ok(M, c.vocab, d, c.dtype, ctx->x_lo != nullptr);
                const TopTable top{ctx->top_table, a.lm_mode == 2 ? 0 : 1};
                ctx->lm_table_rows = table ? M : 0;
                LAUNCH(PROF_GEMM, launch_gemm((char*)ctx->x + off, ctx->x_lo ? (char*)ctx->x_lo + off : nullptr, ctx->lm_head,
                                              lm_out, a.lm_rows, c.vocab, d, c.dtype,
                                              ctx->gemm_ws, ctx->gemm_ws_bytes, st, nullptr, nullptr, gemm_status, table ? &top : nullptr));
            }
        } else if ((s & 1) == 0) {
            char* k_slab = (char*)a.k_cache + ((size_t)l * c.max_batch + a.b0) * seq_stride;
            char* v_slab = (char*)a.v_cache + ((size_t)l * c.max_batch + a.b0) * seq_stride;
            LAUNCH(PROF_ELEMENTWISE, launch_add_rmsnorm(ctx->h, pr, ctx->attn_norm[l], ctx->x, ctx->x_lo, c.dtype, M, d,
                                                        c.rms_eps, st));
            LAUNCH(PROF_GEMM, launch_gemm(ctx->x, ctx->x_lo, ctx->wqkv[l], ctx->y, M, QKV, d, c.dtype, ctx->gemm_ws,
                                          ctx->gemm_ws_bytes, st, &pr, nullptr, gemm_status));
            LAUNCH(PROF_ROPE, launch_rope_kv_write(pr, ctx->inv_freq, a.depth, bt, ctx->q, k_slab, v_slab, c.dtype,
                                                   c.n_heads, Hkv, c.head_dim, c.max_seq, st));
            // inside the decoder the attention result reaches the output projection as a bf16 pair, like every
            // other projection input
            if (!pieces) {
                LAUNCH(PROF_ATTENTION, launch_tree_attention(ctx->q, k_slab, v_slab, a.anc, a.anc_words, bt, c.n_heads, Hkv, c.head_dim,
                                                             c.max_seq, c.dtype, ctx->x, ctx->x_lo, ctx->attn_ws,
                                                             ctx->attn_ws_bytes, st, attn_status));
            } else {
                // the pieces of the chunk are the sequences of ONE launch: piece j sees the prompt so far plus the pieces
                // before it as cached rows (all written by the rotary kernel above, inside this chain) of the same cache
                Batch bj{pieces->lens, pieces->off_pieces, pieces->n, M, pieces->sub, bt.max_len, 0, 1};
                LAUNCH(PROF_ATTENTION, launch_tree_attention(ctx->q, k_slab, v_slab, a.anc, a.anc_words, bj, c.n_heads, Hkv, c.head_dim,
                                                             c.max_seq, c.dtype, ctx->x, ctx->x_lo, ctx->attn_ws,
                                                             ctx->attn_ws_bytes, st, attn_status));
            }
            // While the attention kernel runs, HBM is nearly idle and the SMs it leaves free go to the first CTAs of
            // the output projection, which only wait: they ask for the start of the gate/up weights into L2.
            const WeightPrefetch ahead{ctx->w_gate_up[l], 2 * c.d_ff, d, AHEAD_BYTES, 2 * std::max(0, ctx->sm_count - attn_grid), AHEAD_SELF_BYTES};
            LAUNCH(PROF_GEMM, launch_gemm(ctx->x, ctx->x_lo, ctx->wo[l], ctx->y, M, d, HD, c.dtype, ctx->gemm_ws,
                                          ctx->gemm_ws_bytes, st, out_parts, &ahead, gemm_status));
        } else {
            LAUNCH(PROF_ELEMENTWISE, launch_add_rmsnorm(ctx->h, pr, ctx->mlp_norm[l], ctx->x, ctx->x_lo, c.dtype, M, d,
                                                        c.rms_eps, st));
            LAUNCH(PROF_GEMM, launch_gemm(ctx->x, ctx->x_lo, ctx->w_gate_up[l], ctx->y, M, 2 * c.d_ff, d, c.dtype, ctx->gemm_ws,
                                          ctx->gemm_ws_bytes, st, &pr, nullptr, gemm_status));
            LAUNCH(PROF_ELEMENTWISE, launch_swiglu(pr, ctx->act, ctx->act_lo, c.dtype, M, c.d_ff, st));
            LAUNCH(PROF_GEMM, launch_gemm(ctx->act, ctx->act_lo, ctx->w_down[l], ctx->y, M, d, c.d_ff, c.dtype, ctx->gemm_ws,
                                          ctx->gemm_ws_bytes, st, out_parts, nullptr, gemm_status));
        }
        if (!out_parts) pr = Parts{ctx->y, 1, 0};
    }
    return TRJ_OK;
}

// One forward of the decoder over the rows of `bt`: embedding, then every segment.
trj_status forward(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t b0, const Batch& bt,
                   const int32_t* tokens, const int32_t* depth, const uint64_t* anc, int32_t anc_words,
                   int32_t lm_first, int32_t lm_rows, cudaStream_t st, const SubChunks* pieces = nullptr, int32_t lm_mode = 0) {
    ChainScope chain;                        // the embedding below is the chain's fence
    const trj_model_cfg& c = ctx->cfg;
    LAUNCH(PROF_ELEMENTWISE, launch_embed(ctx->embed, c.dtype, tokens, ctx->h, bt.rows_total, c.d_model, st));
    Parts pr{nullptr, 1, 0};                 // result of the latest projection, possibly in split-K pieces
    const StepArgs a{k_cache, v_cache, b0, bt, tokens, depth, anc, anc_words, lm_first, lm_rows, pieces, lm_mode};
    return run_segments(ctx, a, 0, 2 * c.n_layers + 1, pr, false, st);
}

// Arg-max (and, when asked, acceptance) of the rows the latest forward scored: from the candidates the LM head's
// epilogue left, or from the logits.
cudaError_t step_argmax(trj_ctx* ctx, const int32_t* tokens, const int32_t* parent, const int32_t* depth, const int32_t* row_off,
                        int32_t B, int32_t rows, int32_t* node_argmax, float* margin, int32_t* k_acc, int32_t* path, int32_t* bonus,
                        bool do_accept, cudaStream_t st) {
    if (ctx->lm_table_rows == rows)
        return launch_argmax_table_accept(ctx->top_table, (int32_t)(gemm_top_table_entries(1, ctx->cfg.vocab)), tokens, parent, depth,
                                          row_off, B, rows, node_argmax, margin, k_acc, path, bonus, do_accept, ctx->argmax_ws, st);
    return launch_topk_accept(ctx->logits, TRJ_F32, ctx->cfg.vocab, 1, tokens, parent, depth, row_off, B, rows, nullptr, node_argmax,
                              margin, k_acc, path, bonus, do_accept, ctx->argmax_ws, st);
}

trj_status check_step_args(const trj_ctx* ctx, int32_t B, int32_t rows_total, int32_t max_rows, int32_t max_len,
                           int32_t anc_words) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "null context");
    const trj_model_cfg& c = ctx->cfg;
    TRJ_REQUIRE(B >= 1 && B <= c.max_batch, TRJ_ECAPACITY, "batch %d outside 1..%d", B, c.max_batch);
    TRJ_REQUIRE(max_rows >= 1 && max_rows <= c.max_rows, TRJ_ECAPACITY, "%d rows per tree exceed max_rows %d", max_rows, c.max_rows);
    TRJ_REQUIRE(rows_total >= B && rows_total <= B * max_rows, TRJ_EINVAL, "rows_total %d inconsistent with batch %d x %d", rows_total, B, max_rows);
    TRJ_REQUIRE(max_len >= max_rows && max_len <= c.max_seq, TRJ_ECAPACITY, "max_len %d outside %d..%d", max_len, max_rows, c.max_seq);
    TRJ_REQUIRE(anc_words >= (max_rows + 63) / 64, TRJ_EINVAL, "anc_words %d too small", anc_words);
    return TRJ_OK;
}

}  // namespace

extern "C" size_t trj_workspace_bytes(const trj_model_cfg* cfg) {
    if (check_cfg(cfg) != TRJ_OK) return 0;
    return carve(*cfg, nullptr, nullptr);
}

extern "C" trj_status trj_create(const trj_model_cfg* cfg, const trj_weights* w,
                                 void* workspace, size_t workspace_bytes, trj_ctx** out) {
    TRJ_REQUIRE(out, TRJ_EINVAL, "create: null out");
    *out = nullptr;
    trj_status s = check_cfg(cfg);
    if (s != TRJ_OK) return s;
    TRJ_REQUIRE(w && w->embed && w->lm_head && w->final_norm && w->attn_norm && w->wqkv && w->wo && w->mlp_norm &&
                w->w_gate_up && w->w_down, TRJ_EINVAL, "create: null weight table");
    for (int l = 0; l < cfg->n_layers; ++l)
        TRJ_REQUIRE(w->attn_norm[l] && w->wqkv[l] && w->wo[l] && w->mlp_norm[l] && w->w_gate_up[l] && w->w_down[l],
                    TRJ_EINVAL, "create: null weight in layer %d", l);
    TRJ_REQUIRE(workspace && aligned(workspace, 256), TRJ_EINVAL, "create: workspace must be 256-byte aligned");
    TRJ_REQUIRE(workspace_bytes >= trj_workspace_bytes(cfg), TRJ_ECAPACITY, "create: workspace of %zu bytes, need %zu",
                workspace_bytes, trj_workspace_bytes(cfg));
    trj_ctx* ctx = new (std::nothrow) trj_ctx();
    TRJ_REQUIRE(ctx, TRJ_ECUDA, "create: out of host memory");
    ctx->cfg = *cfg;
    {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            sms = 0;
        ctx->sm_count = sms;
    }
    ctx->embed = w->embed; ctx->lm_head = w->lm_head; ctx->final_norm = w->final_norm;
    for (int l = 0; l < cfg->n_layers; ++l) {
        ctx->attn_norm.push_back(w->attn_norm[l]); ctx->mlp_norm.push_back(w->mlp_norm[l]);
        ctx->wqkv.push_back(w->wqkv[l]); ctx->wo.push_back(w->wo[l]);
        ctx->w_gate_up.push_back(w->w_gate_up[l]); ctx->w_down.push_back(w->w_down[l]);
    }
    carve(*cfg, workspace, ctx);
    ctx->pin_in = ctx->pin_out = nullptr;
    // tables: rotary frequencies and the chain tree used by prefill
    const int half = cfg->head_dim / 2;
    std::vector<double> freq(half);
    for (int i = 0; i < half; ++i) freq[i] = std::pow((double)cfg->rope_theta, -2.0 * i / cfg->head_dim);
    std::vector<int32_t> par(TRJ_MAX_ROWS), dep(TRJ_MAX_ROWS), long_dep(PREFILL_CHUNK);
    for (int i = 0; i < PREFILL_CHUNK; ++i) long_dep[i] = i;
    std::vector<uint64_t> anc(TRJ_MAX_ROWS * 2), anc_long((size_t)PREFILL_CHUNK * 2);
    for (int i = 0; i < TRJ_MAX_ROWS; ++i) par[i] = i - 1;
    tree_from_parents_impl(par.data(), TRJ_MAX_ROWS, 2, dep.data(), anc.data());
    const int piece_rows = std::min(cfg->max_rows, TRJ_MAX_ROWS);
    for (int i = 0; i < PREFILL_CHUNK; ++i) { anc_long[2 * i] = anc[2 * (i % piece_rows)]; anc_long[2 * i + 1] = anc[2 * (i % piece_rows) + 1]; }
    const int32_t unit[2] = {0, 1};
    cudaError_t e = cudaMemcpy(ctx->inv_freq, freq.data(), sizeof(double) * half, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(ctx->chain_depth, long_dep.data(), sizeof(int32_t) * PREFILL_CHUNK, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(ctx->chain_anc, anc_long.data(), sizeof(uint64_t) * PREFILL_CHUNK * 2, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(ctx->unit_row_off, unit, sizeof(unit), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMallocHost((void**)&ctx->pin_in, STEP_IN_BYTES);
    if (e == cudaSuccess) e = cudaMallocHost((void**)&ctx->pin_out, sizeof(int32_t) * STEP_OUT_INTS);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->cap_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->order_ev, cudaEventDisableTiming);
    if (e != cudaSuccess) {
        if (ctx->pin_in) cudaFreeHost(ctx->pin_in);
        if (ctx->pin_out) cudaFreeHost(ctx->pin_out);
        if (ctx->cap_stream) cudaStreamDestroy(ctx->cap_stream);
        if (ctx->order_ev) cudaEventDestroy(ctx->order_ev);
        delete ctx;
        return fail(TRJ_ECUDA, "create: %s", cudaGetErrorString(e));
    }
    *out = ctx;
    return TRJ_OK;
}

extern "C" trj_status trj_destroy(trj_ctx* ctx) {
    if (!ctx) return TRJ_OK;
    if (ctx->pin_in) cudaFreeHost(ctx->pin_in);
    if (ctx->pin_out) cudaFreeHost(ctx->pin_out);
    for (cudaEvent_t e : ctx->prof_ev) cudaEventDestroy(e);
    for (const trj_ctx::GraphEntry& g : ctx->graphs) cudaGraphExecDestroy(g.exec);
    for (const trj_ctx::LoopGraph& g : ctx->loop_graphs) cudaGraphExecDestroy(g.exec);
    if (ctx->cap_stream) cudaStreamDestroy(ctx->cap_stream);
    if (ctx->order_ev) cudaEventDestroy(ctx->order_ev);
    delete ctx;
    return TRJ_OK;
}

extern "C" trj_status trj_device_status(trj_ctx* ctx, int32_t clear, void* stream) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "device_status: null context");
    cudaStream_t st = (cudaStream_t)stream;
    int32_t words[2] = {0, 0};
    TRJ_CHECK_CUDA(cudaMemcpyAsync(words, ctx->dev_status, sizeof(words), cudaMemcpyDeviceToHost, st));
    TRJ_CHECK_CUDA(cudaStreamSynchronize(st));
    if (words[0] == 0 && words[1] == 0) return TRJ_OK;
    if (clear) {
        TRJ_CHECK_CUDA(cudaMemsetAsync(ctx->dev_status, 0, sizeof(words), st));
        TRJ_CHECK_CUDA(cudaStreamSynchronize(st));
    }
    return fail(TRJ_ETIMEOUT, "a bounded device-side wait expired (projection status %d, attention status %d)", words[0], words[1]);
}

extern "C" trj_status trj_selftest_wait_expiry(int32_t* status, int32_t polls, void* stream) {
    TRJ_REQUIRE(status, TRJ_EINVAL, "selftest_wait_expiry: null status word");
    TRJ_REQUIRE(polls >= 1 && polls <= (1 << 21), TRJ_EINVAL, "selftest_wait_expiry: polls %d outside 1..2^21", polls);
    TRJ_CHECK_CUDA(launch_wait_expiry_selftest(status, (uint32_t)polls, (cudaStream_t)stream));
    return TRJ_OK;
}

extern "C" trj_status trj_debug_flags(int32_t* flags) {
#ifdef TRJ_DEBUG
    TRJ_REQUIRE(flags, TRJ_EINVAL, "debug_flags: null pointer");
    int f = 0;
    TRJ_CHECK_CUDA(debug_flags_read(&f));
    *flags = f;
    return TRJ_OK;
#else
    (void)flags;
    return fail(TRJ_EUNSUPPORTED, "debug_flags: this library was built without -DTRJ_DEBUG");
#endif
}

extern "C" trj_status trj_timeline_reset(void* stream) {
#ifdef TRJ_TIMELINE
    cudaStream_t st = (cudaStream_t)stream;
    TRJ_CHECK_CUDA(timeline_reset_generic(st));
    TRJ_CHECK_CUDA(timeline_reset_gemm(st));
    TRJ_CHECK_CUDA(timeline_reset_attention(st));
    return TRJ_OK;
#else
    (void)stream;
    return fail(TRJ_EUNSUPPORTED, "timeline: this library was built without -DTRJ_TIMELINE");
#endif
}

extern "C" trj_status trj_timeline_ctas_per_sm(int32_t* peak) {
#ifdef TRJ_TIMELINE
    TRJ_REQUIRE(peak, TRJ_EINVAL, "timeline_ctas_per_sm: null pointer");
    const int v = timeline_gemm_ctas_per_sm();
    TRJ_REQUIRE(v >= 0, TRJ_ECUDA, "timeline_ctas_per_sm: copy from the device failed");
    *peak = v;
    return TRJ_OK;
#else
    (void)peak;
    return fail(TRJ_EUNSUPPORTED, "timeline: this library was built without -DTRJ_TIMELINE");
#endif
}

extern "C" trj_status trj_timeline_read(int32_t kind, int32_t max_launches, uint64_t* begin_ns, uint64_t* end_ns, int32_t* n_launches) {
#ifdef TRJ_TIMELINE
    TRJ_REQUIRE(begin_ns && end_ns && n_launches && max_launches >= 0, TRJ_EINVAL, "timeline_read: null pointer");
    TRJ_REQUIRE(kind >= 0 && kind < TRJ_TL_KINDS, TRJ_EINVAL, "timeline_read: kind %d outside 0..%d", kind, TRJ_TL_KINDS - 1);
    int n = kind == TRJ_TL_GEMM ? timeline_read_gemm(kind, max_launches, begin_ns, end_ns)
          : kind == TRJ_TL_ATTENTION ? timeline_read_attention(kind, max_launches, begin_ns, end_ns)
                                     : timeline_read_generic(kind, max_launches, begin_ns, end_ns);
    TRJ_REQUIRE(n >= 0, TRJ_ECUDA, "timeline_read: copy from the device failed");
    *n_launches = n;
    return TRJ_OK;
#else
    (void)kind; (void)max_launches; (void)begin_ns; (void)end_ns; (void)n_launches;
    return fail(TRJ_EUNSUPPORTED, "timeline: this library was built without -DTRJ_TIMELINE");
#endif
}

extern "C" uint64_t trj_launch_count(void) { return launches_so_far(); }
extern "C" void trj_set_pdl(int32_t on) { set_pdl(on != 0); }

extern "C" trj_status trj_profile_enable(trj_ctx* ctx, int32_t on) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "profile_enable: null context");
    if (on && ctx->prof_ev.empty()) {
        ctx->prof_ev.resize(2 * PROF_MAX_LAUNCHES);
        ctx->prof_cat.resize(PROF_MAX_LAUNCHES);
        for (cudaEvent_t& e : ctx->prof_ev) TRJ_CHECK_CUDA(cudaEventCreate(&e));
    }
    ctx->prof_on = on != 0;
    ctx->prof_used = 0;
    return TRJ_OK;
}

extern "C" trj_status trj_profile_read(trj_ctx* ctx, float* ms, int32_t* launches, int32_t keep) {
    TRJ_REQUIRE(ctx && ms && launches, TRJ_EINVAL, "profile_read: null pointer");
    for (int c = 0; c < TRJ_PROF_CATEGORIES; ++c) { ms[c] = 0.f; launches[c] = 0; }
    for (size_t i = 0; i < ctx->prof_used; ++i) {
        TRJ_CHECK_CUDA(cudaEventSynchronize(ctx->prof_ev[2 * i + 1]));
        float t = 0.f;
        TRJ_CHECK_CUDA(cudaEventElapsedTime(&t, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]));
        ms[ctx->prof_cat[i]] += t;
        launches[ctx->prof_cat[i]] += 1;
    }
    if (!keep) ctx->prof_used = 0;
    return TRJ_OK;
}

extern "C" trj_status trj_verify_step(trj_ctx* ctx, void* k_cache, void* v_cache, const int32_t* seq_len,
                                      const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                      const uint64_t* anc, int32_t anc_words, const int32_t* row_off,
                                      int32_t B, int32_t rows_total, int32_t max_rows, int32_t max_len,
                                      int32_t* node_argmax, float* margin, float* logits, void* stream) {
    trj_status s = check_step_args(ctx, B, rows_total, max_rows, max_len, anc_words);
    if (s != TRJ_OK) return s;
    TRJ_REQUIRE(k_cache && v_cache && seq_len && tokens && parent && depth && anc && row_off && node_argmax,
                TRJ_EINVAL, "verify_step: null pointer");
    cudaStream_t st = (cudaStream_t)stream;
    ChainScope chain;
    Batch bt{seq_len, row_off, B, rows_total, max_rows, max_len};
    // the logits stay materialised: the caller may ask for them here or for their top-K afterwards (trj_node_topk)
    s = forward(ctx, k_cache, v_cache, 0, bt, tokens, depth, anc, anc_words, 0, rows_total, st, nullptr, 1);
    if (s != TRJ_OK) return s;
    LAUNCH(PROF_ARGMAX, step_argmax(ctx, tokens, parent, depth, row_off, B, rows_total, node_argmax, margin, nullptr, nullptr, nullptr,
                                    false, st));
    ctx->last_rows = rows_total; ctx->last_row_off = row_off; ctx->last_B = B;
    if (logits)
        TRJ_CHECK_CUDA(cudaMemcpyAsync(logits, ctx->logits, sizeof(float) * (size_t)rows_total * ctx->cfg.vocab,
                                       cudaMemcpyDeviceToDevice, st));
    return TRJ_OK;
}

// ---- tensor-parallel stepping: one context per rank, each holding a slice of the heads and of the feed-forward
// width.  Every half of a layer ends in a projection whose result is a partial sum over the rank's slice; the
// caller adds the ranks' partial sums (the exchange buffer) between two segments.
extern "C" int32_t trj_tp_segments(const trj_ctx* ctx) { return ctx ? 2 * ctx->cfg.n_layers + 1 : 0; }

extern "C" trj_status trj_tp_begin(trj_ctx* ctx, void* k_cache, void* v_cache, const int32_t* seq_len,
                                   const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                   const uint64_t* anc, int32_t anc_words, const int32_t* row_off,
                                   int32_t B, int32_t rows_total, int32_t max_rows, int32_t max_len, void* stream) {
    trj_status s = check_step_args(ctx, B, rows_total, max_rows, max_len, anc_words);
    if (s != TRJ_OK) return s;
    TRJ_REQUIRE(k_cache && v_cache && seq_len && tokens && parent && depth && anc && row_off, TRJ_EINVAL, "tp_begin: null pointer");
    cudaStream_t st = (cudaStream_t)stream;
    ChainScope chain;
    ctx->tp = trj_ctx::TpStep{};
    LAUNCH(PROF_ELEMENTWISE, launch_embed(ctx->embed, ctx->cfg.dtype, tokens, ctx->h, rows_total, ctx->cfg.d_model, st));
    ctx->tp.open = true; ctx->tp.next = 0; ctx->tp.k_cache = k_cache; ctx->tp.v_cache = v_cache;
    ctx->tp.bt = Batch{seq_len, row_off, B, rows_total, max_rows, max_len};
    ctx->tp.tokens = tokens; ctx->tp.parent = parent; ctx->tp.depth = depth; ctx->tp.anc = anc; ctx->tp.anc_words = anc_words;
    return TRJ_OK;
}

extern "C" trj_status trj_tp_segment(trj_ctx* ctx, int32_t segment, void* stream) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "tp_segment: null context");
    TRJ_REQUIRE(ctx->tp.open, TRJ_EINVAL, "tp_segment: no step begun");
    const int32_t n_seg = 2 * ctx->cfg.n_layers + 1;
    TRJ_REQUIRE(segment == ctx->tp.next && segment < n_seg, TRJ_EINVAL, "tp_segment: segment %d asked, %d is next of %d",
                segment, ctx->tp.next, n_seg);
    cudaStream_t st = (cudaStream_t)stream;
    ChainScope chain;
    const trj_ctx::TpStep& t = ctx->tp;
    const StepArgs a{t.k_cache, t.v_cache, 0, t.bt, t.tokens, t.depth, t.anc, t.anc_words, 0, t.bt.rows_total, nullptr, 0};
    // what the previous segment left, summed over the ranks by the caller, sits in the exchange buffer
    Parts pr = segment == 0 ? Parts{nullptr, 1, 0} : whole(ctx->y);
    trj_status s = run_segments(ctx, a, segment, segment + 1, pr, segment + 1 < n_seg, st);
    if (s != TRJ_OK) { ctx->tp.open = false; return s; }
    ctx->tp.next = segment + 1;
    return TRJ_OK;
}

extern "C" trj_status trj_tp_exchange_buffer(const trj_ctx* ctx, float** partial, size_t* count) {
    TRJ_REQUIRE(ctx && partial && count, TRJ_EINVAL, "tp_exchange_buffer: null pointer");
    TRJ_REQUIRE(ctx->tp.open, TRJ_EINVAL, "tp_exchange_buffer: no step begun");
    *partial = ctx->y;
    *count = (size_t)ctx->tp.bt.rows_total * ctx->cfg.d_model;
    return TRJ_OK;
}

extern "C" trj_status trj_tp_finish(trj_ctx* ctx, int32_t* node_argmax, float* margin, float* logits, void* stream) {
    TRJ_REQUIRE(ctx && node_argmax, TRJ_EINVAL, "tp_finish: null pointer");
    const int32_t n_seg = 2 * ctx->cfg.n_layers + 1;
    TRJ_REQUIRE(ctx->tp.open && ctx->tp.next == n_seg, TRJ_EINVAL, "tp_finish: %d of %d segments run",
                ctx->tp.open ? ctx->tp.next : 0, n_seg);
    cudaStream_t st = (cudaStream_t)stream;
    ChainScope chain;
    const trj_ctx::TpStep& t = ctx->tp;
    const int32_t rows = t.bt.rows_total;
    LAUNCH(PROF_ARGMAX, launch_topk_accept(ctx->logits, TRJ_F32, ctx->cfg.vocab, 1, t.tokens, t.parent, t.depth, t.bt.row_off, t.bt.B,
                                           rows, nullptr, node_argmax, margin, nullptr, nullptr, nullptr, false,
                                           ctx->argmax_ws, st));
    ctx->last_rows = rows; ctx->last_row_off = t.bt.row_off; ctx->last_B = t.bt.B;
    ctx->tp.open = false;
    if (logits)
        TRJ_CHECK_CUDA(cudaMemcpyAsync(logits, ctx->logits, sizeof(float) * (size_t)rows * ctx->cfg.vocab,
                                       cudaMemcpyDeviceToDevice, st));
    return TRJ_OK;
}

extern "C" trj_status trj_node_topk(trj_ctx* ctx, int32_t rows_total, int32_t K, int32_t* topk, void* stream) {
    TRJ_REQUIRE(ctx && topk, TRJ_EINVAL, "node_topk: null pointer");
    TRJ_REQUIRE(K >= 1 && K <= TRJ_MAX_TOPK && K <= ctx->cfg.vocab, TRJ_EINVAL, "node_topk: K = %d outside 1..%d", K, TRJ_MAX_TOPK);
    TRJ_REQUIRE(ctx->last_rows > 0 && rows_total == ctx->last_rows, TRJ_EINVAL,
                "node_topk: %d rows asked, the latest verify_step scored %d", rows_total, ctx->last_rows);
    cudaStream_t st = (cudaStream_t)stream;
    ChainScope chain;
    // predictions and margins are recomputed into scratch of the context (the caller already has them)
    int32_t* scratch_pred = (int32_t*)ctx->y;
    LAUNCH(PROF_ARGMAX, launch_topk_accept(ctx->logits, TRJ_F32, ctx->cfg.vocab, K, nullptr, nullptr, nullptr, ctx->last_row_off,
                                           ctx->last_B, rows_total, topk, scratch_pred, nullptr, nullptr, nullptr, nullptr, false,
                                           ctx->argmax_ws, st));
    return TRJ_OK;
}

extern "C" trj_status trj_accept(trj_ctx* ctx, const int32_t* tokens, const int32_t* parent, const int32_t* depth,
                                 const int32_t* row_off, int32_t B, int32_t rows_total, const int32_t* node_argmax,
                                 int32_t* k_acc, int32_t* path, int32_t* bonus, void* stream) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "accept: null context");
    TRJ_REQUIRE(tokens && parent && depth && row_off && node_argmax && k_acc && path && bonus, TRJ_EINVAL, "accept: null pointer");
    TRJ_REQUIRE(B >= 1 && B <= ctx->cfg.max_batch && rows_total >= B, TRJ_ECAPACITY, "accept: bad batch");
    TRJ_REQUIRE(rows_total <= B * TRJ_MAX_ROWS, TRJ_ECAPACITY, "accept: %d rows in %d trees: a tree holds at most %d rows",
                rows_total, B, TRJ_MAX_ROWS);
    cudaStream_t st = (cudaStream_t)stream;
    ChainScope chain;                        // these kernels wait for their predecessor before reading anything
    LAUNCH(PROF_ARGMAX, launch_argmax_accept(nullptr, TRJ_F32, 0, tokens, parent, depth, row_off, B, rows_total,
                                             const_cast<int32_t*>(node_argmax), nullptr, k_acc, path, bonus, false, true,
                                             ctx->argmax_ws, st));
    return TRJ_OK;
}

extern "C" trj_status trj_compact_kv(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t B,
                                     const int32_t* k_acc, const int32_t* path, void* stream) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "compact_kv: null context");
    TRJ_REQUIRE(k_cache && v_cache && seq_len && k_acc && path, TRJ_EINVAL, "compact_kv: null pointer");
    const trj_model_cfg& c = ctx->cfg;
    TRJ_REQUIRE(B >= 1 && B <= c.max_batch, TRJ_ECAPACITY, "compact_kv: batch %d outside 1..%d", B, c.max_batch);
    cudaStream_t st = (cudaStream_t)stream;
    ChainScope chain;
    LAUNCH(PROF_COMPACT, launch_compact(k_cache, v_cache, c.n_layers, c.max_batch, B, kv_heads(c), c.max_seq, c.head_dim,
                                        c.dtype, seq_len, k_acc, path, st, ctx->compact_tickets));
    return TRJ_OK;
}

extern "C" trj_status trj_prefill(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t b,
                                  const int32_t* tokens, int32_t n, int32_t* first_token, void* stream) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "prefill: null context");
    const trj_model_cfg& c = ctx->cfg;
    TRJ_REQUIRE(k_cache && v_cache && seq_len && tokens && first_token, TRJ_EINVAL, "prefill: null pointer");
    TRJ_REQUIRE(b >= 0 && b < c.max_batch, TRJ_EINVAL, "prefill: sequence %d outside the cache", b);
    TRJ_REQUIRE(n >= 1 && n <= c.max_seq, TRJ_ECAPACITY, "prefill: %d tokens do not fit %d cache rows", n, c.max_seq);
    cudaStream_t st = (cudaStream_t)stream;
    const int32_t sub = std::min(c.max_rows, TRJ_MAX_ROWS);                  // rows of an attention piece
    const int32_t chunk_cap = std::min(PREFILL_CHUNK, PREFILL_MAX_SUB * sub);
    int32_t* lens = ctx->prefill_geo, *off_all = lens + PREFILL_MAX_SUB, *off_pieces = off_all + 2;
    for (int32_t done = 0; done < n; done += chunk_cap) {
        const int32_t m = std::min(chunk_cap, n - done);
        const bool last = done + m >= n;
        const int32_t n_sub = (m + sub - 1) / sub;
        TRJ_CHECK_CUDA(launch_prefill_geometry(seq_len + b, lens, n_sub, sub, m, off_all, off_pieces, st));
        Batch bt{seq_len + b, off_all, 1, m, sub, c.max_seq};
        const SubChunks pieces{n_sub, sub, lens, off_pieces};
        trj_status s = forward(ctx, k_cache, v_cache, b, bt, tokens + done, ctx->chain_depth, ctx->chain_anc, 2,
                               m - 1, last ? 1 : 0, st, &pieces);
        if (s != TRJ_OK) return s;
        if (last)   // greedy prediction after the last prompt token: a one-row arg-max
            TRJ_CHECK_CUDA(launch_topk_accept(ctx->logits, TRJ_F32, c.vocab, 1, nullptr, nullptr,
                                              nullptr, ctx->unit_row_off, 1, 1, nullptr, first_token, nullptr, nullptr,
                                              nullptr, nullptr, false, ctx->argmax_ws, st));
        TRJ_CHECK_CUDA(launch_bump_len(seq_len + b, m, st));
    }
    return TRJ_OK;
}

namespace {

// Everything trj_step_host puts on a stream between the host-side tree build and the final synchronise.
trj_status enqueue_step(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t M, int32_t max_len,
                        cudaStream_t st) {
    const trj_model_cfg& c = ctx->cfg;
    ChainScope chain;
    TRJ_CHECK_CUDA(cudaMemcpyAsync(ctx->step_in, ctx->pin_in, STEP_IN_BYTES, cudaMemcpyHostToDevice, st));
    int32_t* d_tokens = ctx->step_in, *d_parent = d_tokens + TRJ_MAX_ROWS, *d_depth = d_tokens + 2 * TRJ_MAX_ROWS;
    int32_t* d_off = d_tokens + 3 * TRJ_MAX_ROWS;
    uint64_t* d_anc = (uint64_t*)(d_tokens + STEP_IN_INTS);
    int32_t* d_pred = ctx->step_out, *d_k = d_pred + TRJ_MAX_ROWS, *d_bonus = d_k + 1, *d_path = d_k + 2;
    Batch bt{seq_len, d_off, 1, M, M, max_len};
    trj_status s = forward(ctx, k_cache, v_cache, 0, bt, d_tokens, d_depth, d_anc, 2, 0, M, st, nullptr, 2);   // nobody reads this step's logits
    if (s != TRJ_OK) return s;
    LAUNCH(PROF_ARGMAX, step_argmax(ctx, d_tokens, d_parent, d_depth, d_off, 1, M, d_pred, nullptr, d_k, d_path, d_bonus, true, st));
    LAUNCH(PROF_COMPACT, launch_compact(k_cache, v_cache, c.n_layers, c.max_batch, 1, kv_heads(c), c.max_seq, c.head_dim,
                                        c.dtype, seq_len, d_k, d_path, st, ctx->compact_tickets));
    TRJ_CHECK_CUDA(cudaMemcpyAsync(ctx->pin_out, ctx->step_out, sizeof(int32_t) * STEP_OUT_INTS, cudaMemcpyDeviceToHost, st));
    return TRJ_OK;
}

// The launch sequence of a step depends only on the tree size, the attention grid and the buffer addresses,
// so after the first (plain) step it is captured once per such key and replayed as a CUDA graph.
trj_status run_step(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t M, int32_t max_len,
                    cudaStream_t st) {
    const int grid = tree_attention_grid(1, ctx->cfg.n_heads, max_len);
    if (ctx->prof_on || ctx->steps_done == 0 || !ctx->cap_stream) {
        trj_status s = enqueue_step(ctx, k_cache, v_cache, seq_len, M, max_len, st);
        if (s != TRJ_OK) return s;
        TRJ_CHECK_CUDA(cudaStreamSynchronize(st));
        return TRJ_OK;
    }
    cudaGraphExec_t exec = nullptr;
    for (const trj_ctx::GraphEntry& g : ctx->graphs)
        if (g.M == M && g.grid == grid && g.k == k_cache && g.v == v_cache && g.len == seq_len) exec = g.exec;
    if (!exec) {
        cudaGraph_t graph = nullptr;
        TRJ_CHECK_CUDA(cudaStreamBeginCapture(ctx->cap_stream, cudaStreamCaptureModeThreadLocal));
        trj_status s = enqueue_step(ctx, k_cache, v_cache, seq_len, M, max_len, ctx->cap_stream);
        cudaError_t e = cudaStreamEndCapture(ctx->cap_stream, &graph);
        if (s != TRJ_OK) { if (graph) cudaGraphDestroy(graph); return s; }
        if (e != cudaSuccess) return fail(TRJ_ECUDA, "step_host: graph capture: %s", cudaGetErrorString(e));
        e = cudaGraphInstantiate(&exec, graph, 0);
        cudaGraphDestroy(graph);
        if (e != cudaSuccess) return fail(TRJ_ECUDA, "step_host: graph instantiate: %s", cudaGetErrorString(e));
        if (ctx->graphs.size() >= 32) { cudaGraphExecDestroy(ctx->graphs.front().exec); ctx->graphs.erase(ctx->graphs.begin()); }
        ctx->graphs.push_back({M, grid, k_cache, v_cache, seq_len, exec});
    }
    // launched on the caller's stream: the graph runs after everything already enqueued on it
    TRJ_CHECK_CUDA(cudaGraphLaunch(exec, st));
    TRJ_CHECK_CUDA(cudaStreamSynchronize(st));
    return TRJ_OK;
}

}  // namespace

extern "C" trj_status trj_step_host(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t max_len,
                                    int32_t root, const int32_t* window, int32_t W,
                                    const int32_t* branches, int32_t R, int32_t branch_len,
                                    int32_t* tokens, int32_t* parent, int32_t* n_rows, int32_t* node_argmax,
                                    int32_t* k_acc, int32_t* path, int32_t* bonus, void* stream) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "step_host: null context");
    TRJ_REQUIRE(k_cache && v_cache && seq_len && tokens && parent && n_rows && node_argmax && k_acc && path && bonus,
                TRJ_EINVAL, "step_host: null pointer");
    const trj_model_cfg& c = ctx->cfg;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t* in = ctx->pin_in;
    int32_t* h_tokens = in, *h_parent = in + TRJ_MAX_ROWS, *h_depth = in + 2 * TRJ_MAX_ROWS, *h_off = in + 3 * TRJ_MAX_ROWS;
    uint64_t* h_anc = (uint64_t*)(in + STEP_IN_INTS);
    int32_t M = 0;
    trj_status s = trj_build_tree(root, window, W, branches, R, branch_len, c.max_rows, 2, h_tokens, h_parent, h_depth, h_anc, &M);
    if (s != TRJ_OK) return s;
    s = check_step_args(ctx, 1, M, M, max_len, 2);
    if (s != TRJ_OK) return s;
    h_off[0] = 0; h_off[1] = M;
    s = run_step(ctx, k_cache, v_cache, seq_len, M, max_len, st);
    if (s != TRJ_OK) return s;
    ++ctx->steps_done;
    std::memcpy(tokens, h_tokens, sizeof(int32_t) * M);
    std::memcpy(parent, h_parent, sizeof(int32_t) * M);
    *n_rows = M;
    std::memcpy(node_argmax, ctx->pin_out, sizeof(int32_t) * M);
    if (ctx->pin_out[STEP_STATUS_AT] != 0 || ctx->pin_out[STEP_STATUS_AT + 1] != 0) {
        // the words stay set on the device (see trj_device_status); the step's results are not to be trusted
        return fail(TRJ_ETIMEOUT, "step_host: a bounded device-side wait expired (projection status %d, attention status %d)",
                    ctx->pin_out[STEP_STATUS_AT], ctx->pin_out[STEP_STATUS_AT + 1]);
    }
    *k_acc = ctx->pin_out[TRJ_MAX_ROWS];
    *bonus = ctx->pin_out[TRJ_MAX_ROWS + 1];
    std::memcpy(path, ctx->pin_out + TRJ_MAX_ROWS + 2, sizeof(int32_t) * TRJ_PATH_STRIDE);
    return TRJ_OK;
}


// ---------------------------------------------------------------- device-resident drafting, commit and decode loop
extern "C" trj_status trj_draft_tokens(const int32_t* context, const int32_t* n_ctx, const int32_t* window, int32_t W,
                                       int32_t R, int32_t branch_len, const int64_t* draws, int32_t* tokens, void* stream) {
    TRJ_REQUIRE(context && n_ctx && tokens, TRJ_EINVAL, "draft_tokens: null pointer");
    TRJ_REQUIRE(W >= 0 && R >= 0 && branch_len >= 0, TRJ_EINVAL, "draft_tokens: negative size");
    TRJ_REQUIRE(W == 0 || window, TRJ_EINVAL, "draft_tokens: null window");
    TRJ_REQUIRE(R * branch_len == 0 || draws, TRJ_EINVAL, "draft_tokens: null draws");
    TRJ_REQUIRE(R <= 64 && 1 + (int64_t)W + (int64_t)R * branch_len <= TRJ_MAX_ROWS, TRJ_ECAPACITY,
                "draft_tokens: %d + %d x %d draft rows exceed the limits (64 branches, %d rows)", W, R, branch_len, TRJ_MAX_ROWS);
    TRJ_CHECK_CUDA(launch_draft_tokens(context, n_ctx, window, W, R, branch_len, draws, nullptr, tokens, (cudaStream_t)stream));
    return TRJ_OK;
}

extern "C" trj_status trj_commit_refill(const int32_t* tokens, const int32_t* parent, const int32_t* node_argmax, int32_t M,
                                        const int32_t* k_acc, const int32_t* path, const int32_t* bonus, int32_t* context,
                                        int32_t capacity, int32_t* n_ctx, int32_t W, const int64_t* draws, int32_t* window,
                                        int32_t* overflow, void* stream) {
    TRJ_REQUIRE(tokens && parent && node_argmax && k_acc && path && bonus && context && n_ctx, TRJ_EINVAL, "commit_refill: null pointer");
    TRJ_REQUIRE(M >= 1 && M <= TRJ_MAX_ROWS, TRJ_ECAPACITY, "commit_refill: %d rows outside 1..%d", M, TRJ_MAX_ROWS);
    TRJ_REQUIRE(W >= 0 && (W == 0 || (window && draws)), TRJ_EINVAL, "commit_refill: null window or draws");
    TRJ_REQUIRE(capacity >= 1, TRJ_EINVAL, "commit_refill: empty context buffer");
    TRJ_CHECK_CUDA(launch_commit_refill(tokens, parent, node_argmax, M, k_acc, path, bonus, context, capacity, n_ctx, W, W,
                                        draws, nullptr, window, nullptr, overflow, (cudaStream_t)stream));
    return TRJ_OK;
}

extern "C" trj_status trj_set_draft_source(trj_ctx* ctx, const int32_t* stream, int32_t n, const int32_t* take, int32_t n_steps) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "set_draft_source: null context");
    if (!stream) { ctx->draft_src = DraftSource{nullptr, 0, nullptr}; ctx->draft_src_steps = 0; return TRJ_OK; }
    TRJ_REQUIRE(take && n >= 0 && n_steps >= 0, TRJ_EINVAL, "set_draft_source: null take or negative size");
    ctx->draft_src = DraftSource{stream, n, take};
    ctx->draft_src_steps = n_steps;
    return TRJ_OK;
}

namespace {

// Runs n_steps of a device-resident decode loop whose single step `enqueue_one` puts on a stream.  The first step a
// context ever runs is enqueued plainly (one-time set-up of the kernels happens outside any capture); so is
// everything while profiling or without a capture stream.  Otherwise one step is captured once per key (every
// pointer and size the step depends on) and the graph is launched once per step: the device step counter makes the
// steps differ.
template <typename EnqueueOne>
trj_status run_device_loop(trj_ctx* ctx, const std::vector<uint64_t>& key, int32_t n_steps, EnqueueOne&& enqueue_one, cudaStream_t st) {
    trj_status s = TRJ_OK;
    int32_t done = 0;
    const bool plain = ctx->prof_on || !ctx->cap_stream;
    if (ctx->steps_done == 0 || plain) {
        const int32_t n_plain = plain ? n_steps : 1;
        for (; done < n_plain; ++done) {
            s = enqueue_one(st);
            if (s != TRJ_OK) return s;
        }
    }
    if (done < n_steps) {
        cudaGraphExec_t exec = nullptr;
        for (const trj_ctx::LoopGraph& g : ctx->loop_graphs)
            if (g.key == key) exec = g.exec;
        if (!exec) {
            cudaGraph_t graph = nullptr;
            TRJ_CHECK_CUDA(cudaStreamBeginCapture(ctx->cap_stream, cudaStreamCaptureModeThreadLocal));
            s = enqueue_one(ctx->cap_stream);
            cudaError_t e = cudaStreamEndCapture(ctx->cap_stream, &graph);
            if (s != TRJ_OK) { if (graph) cudaGraphDestroy(graph); return s; }
            if (e != cudaSuccess) return fail(TRJ_ECUDA, "decode loop: graph capture: %s", cudaGetErrorString(e));
            e = cudaGraphInstantiate(&exec, graph, 0);
            cudaGraphDestroy(graph);
            if (e != cudaSuccess) return fail(TRJ_ECUDA, "decode loop: graph instantiate: %s", cudaGetErrorString(e));
            if (ctx->loop_graphs.size() >= 8) { cudaGraphExecDestroy(ctx->loop_graphs.front().exec); ctx->loop_graphs.erase(ctx->loop_graphs.begin()); }
            ctx->loop_graphs.push_back({key, exec});
        }
        for (; done < n_steps; ++done) TRJ_CHECK_CUDA(cudaGraphLaunch(exec, st));
    }
    ctx->steps_done += n_steps;
    return TRJ_OK;
}

}  // namespace

extern "C" trj_status trj_decode_device(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t* context,
                                        int32_t capacity, int32_t* n_ctx, int32_t n_ctx_now, int32_t* window, int32_t W,
                                        int32_t R, int32_t branch_len, const int64_t* draws, int32_t n_steps,
                                        int32_t* k_log, void* stream) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "decode_device: null context");
    TRJ_REQUIRE(k_cache && v_cache && seq_len && context && n_ctx && draws, TRJ_EINVAL, "decode_device: null pointer");
    TRJ_REQUIRE(W >= 0 && R >= 0 && branch_len >= 0 && n_steps >= 0 && (W == 0 || window), TRJ_EINVAL, "decode_device: bad sizes");
    const trj_model_cfg& c = ctx->cfg;
    const int64_t M64 = 1 + (int64_t)W + (int64_t)R * branch_len;
    TRJ_REQUIRE(R <= 64 && M64 <= c.max_rows, TRJ_ECAPACITY, "decode_device: %lld tree rows exceed max_rows %d (or more than 64 branches)",
                (long long)M64, c.max_rows);
    const int32_t M = (int32_t)M64;
    // a step commits at most depth + 1 tokens; the deepest node is the end of the window chain or of a branch
    const int32_t per_step = std::max(W, branch_len) + 1;
    TRJ_REQUIRE(n_ctx_now >= 1, TRJ_EINVAL, "decode_device: empty context");
    TRJ_REQUIRE((int64_t)n_ctx_now + (int64_t)n_steps * per_step <= capacity, TRJ_ECAPACITY,
                "decode_device: context buffer of %d cannot take %d steps of up to %d tokens after %d", capacity, n_steps, per_step, n_ctx_now);
    // the cache holds every committed token but the last one (the next root) and, during a step, the tree rows
    const int64_t max_len = (int64_t)n_ctx_now - 1 + (int64_t)n_steps * per_step + M;
    TRJ_REQUIRE(max_len <= c.max_seq, TRJ_ECAPACITY, "decode_device: up to %lld cache rows exceed max_seq %d", (long long)max_len, c.max_seq);
    TRJ_REQUIRE(!ctx->draft_src.stream || ctx->draft_src_steps >= n_steps, TRJ_ECAPACITY,
                "decode_device: the draft source covers %d steps, %d asked", ctx->draft_src_steps, n_steps);
    trj_status s = check_step_args(ctx, 1, M, M, (int32_t)max_len, 2);
    if (s != TRJ_OK) return s;
    if (n_steps == 0) return TRJ_OK;
    cudaStream_t st = (cudaStream_t)stream;
    // the tree's shape is static: parents, depths, ancestor masks and row offsets go to the device once
    int32_t* in = ctx->pin_in;
    int32_t* h_tokens = in, *h_parent = in + TRJ_MAX_ROWS, *h_depth = in + 2 * TRJ_MAX_ROWS, *h_off = in + 3 * TRJ_MAX_ROWS;
    uint64_t* h_anc = (uint64_t*)(in + STEP_IN_INTS);
    {
        std::vector<int32_t> zeros((size_t)std::max(W, R * branch_len) + 1, 0);
        int32_t m_built = 0;
        s = trj_build_tree(0, zeros.data(), W, zeros.data(), R, branch_len, c.max_rows, 2, h_tokens, h_parent, h_depth, h_anc, &m_built);
        if (s != TRJ_OK) return s;
    }
    h_off[0] = 0; h_off[1] = M;
    TRJ_CHECK_CUDA(cudaMemcpyAsync(ctx->step_in, ctx->pin_in, STEP_IN_BYTES, cudaMemcpyHostToDevice, st));
    TRJ_CHECK_CUDA(cudaMemsetAsync(ctx->loop_state, 0, sizeof(int32_t) * 64, st));
    // the pinned staging area is shared with trj_step_host: the copy must have left it before this call returns
    TRJ_CHECK_CUDA(cudaEventRecord(ctx->order_ev, st));
    TRJ_CHECK_CUDA(cudaEventSynchronize(ctx->order_ev));
    int32_t* d_tokens = ctx->step_in, *d_parent = d_tokens + TRJ_MAX_ROWS, *d_depth = d_tokens + 2 * TRJ_MAX_ROWS;
    int32_t* d_off = d_tokens + 3 * TRJ_MAX_ROWS;
    uint64_t* d_anc = (uint64_t*)(d_tokens + STEP_IN_INTS);
    int32_t* d_pred = ctx->step_out, *d_k = d_pred + TRJ_MAX_ROWS, *d_bonus = d_k + 1, *d_path = d_k + 2;
    int32_t* d_step = ctx->loop_state, *d_overflow = ctx->loop_state + 1;
    Batch bt{seq_len, d_off, 1, M, M, (int32_t)max_len};
    auto enqueue_one = [&](cudaStream_t on) -> trj_status {
        ChainScope chain;
        LAUNCH_ON(on, PROF_ELEMENTWISE, launch_draft_tokens(context, n_ctx, window, W, R, branch_len, draws, d_step, d_tokens, on,
                                                            ctx->draft_src));
        trj_status fs = forward(ctx, k_cache, v_cache, 0, bt, d_tokens, d_depth, d_anc, 2, 0, M, on, nullptr, 2);
        if (fs != TRJ_OK) return fs;
        LAUNCH_ON(on, PROF_ARGMAX, step_argmax(ctx, d_tokens, d_parent, d_depth, d_off, 1, M, d_pred, nullptr, d_k, d_path, d_bonus, true, on));
        LAUNCH_ON(on, PROF_COMPACT, launch_compact(k_cache, v_cache, c.n_layers, c.max_batch, 1, kv_heads(c), c.max_seq, c.head_dim,
                                                   c.dtype, seq_len, d_k, d_path, on, ctx->compact_tickets));
        LAUNCH_ON(on, PROF_ELEMENTWISE, launch_commit_refill(d_tokens, d_parent, d_pred, M, d_k, d_path, d_bonus, context, capacity,
                                                             n_ctx, W, W + R * branch_len, draws, d_step, window, k_log, d_overflow, on));
        return TRJ_OK;
    };
    const std::vector<uint64_t> key_of_loop = {(uint64_t)0 /* window + branches */, (uint64_t)M, (uint64_t)tree_attention_grid(1, c.n_heads, (int32_t)max_len),
                                           (uint64_t)(uintptr_t)k_cache, (uint64_t)(uintptr_t)v_cache, (uint64_t)(uintptr_t)seq_len,
                                           (uint64_t)(uintptr_t)context, (uint64_t)capacity, (uint64_t)(uintptr_t)n_ctx,
                                           (uint64_t)(uintptr_t)window, (uint64_t)W, (uint64_t)R, (uint64_t)branch_len,
                                           (uint64_t)(uintptr_t)draws, (uint64_t)(uintptr_t)k_log, (uint64_t)max_len,
                                           (uint64_t)(uintptr_t)ctx->draft_src.stream, (uint64_t)ctx->draft_src.n,
                                           (uint64_t)(uintptr_t)ctx->draft_src.take};
    return run_device_loop(ctx, key_of_loop, n_steps, enqueue_one, st);
}

extern "C" trj_status trj_decode_device_tree(trj_ctx* ctx, void* k_cache, void* v_cache, int32_t* seq_len, int32_t* context,
                                             int32_t capacity, int32_t* n_ctx, int32_t n_ctx_now, const int32_t* parent,
                                             const int32_t* rank, int32_t M, int32_t K, int32_t n_retrieved, int32_t* drafts,
                                             const int64_t* draws, int32_t n_steps, int32_t* k_log, void* stream) {
    TRJ_REQUIRE(ctx, TRJ_EINVAL, "decode_device_tree: null context");
    TRJ_REQUIRE(k_cache && v_cache && seq_len && context && n_ctx && parent && rank && draws, TRJ_EINVAL, "decode_device_tree: null pointer");
    const trj_model_cfg& c = ctx->cfg;
    TRJ_REQUIRE(M >= 1 && M <= c.max_rows && M <= TRJ_MAX_ROWS, TRJ_ECAPACITY, "decode_device_tree: %d tree rows outside 1..%d", M, c.max_rows);
    TRJ_REQUIRE(M == 1 || drafts, TRJ_EINVAL, "decode_device_tree: null drafts");
    TRJ_REQUIRE(K >= 1 && K <= TRJ_MAX_TOPK && K <= c.vocab, TRJ_EINVAL, "decode_device_tree: K = %d outside 1..%d", K, TRJ_MAX_TOPK);
    TRJ_REQUIRE(n_retrieved >= 0 && n_retrieved < TRJ_MAX_ROWS && n_steps >= 0, TRJ_EINVAL, "decode_device_tree: bad sizes");
    // the template on the host: depths, ancestor masks, and what the device kernels rely on without checking
    int32_t* in = ctx->pin_in;
    int32_t* h_parent = in + TRJ_MAX_ROWS, *h_depth = in + 2 * TRJ_MAX_ROWS, *h_off = in + 3 * TRJ_MAX_ROWS;
    uint64_t* h_anc = (uint64_t*)(in + STEP_IN_INTS);
    TRJ_REQUIRE(parent[0] == -1, TRJ_EINVAL, "decode_device_tree: row 0 must be the root");
    for (int32_t i = 1; i < M; ++i)
        TRJ_REQUIRE(parent[i] >= 0 && parent[i] < i, TRJ_EINVAL, "decode_device_tree: parent[%d] = %d is not an earlier row", i, parent[i]);
    for (int32_t i = 0; i < M; ++i) h_parent[i] = parent[i];
    trj_status s = tree_from_parents_impl(h_parent, M, 2, h_depth, h_anc);
    if (s != TRJ_OK) return s;
    int32_t deepest = 0;
    for (int32_t i = 1; i < M; ++i) {
        deepest = std::max(deepest, h_depth[i]);
        TRJ_REQUIRE(rank[i] >= 0 ? rank[i] < K : -1 - rank[i] < n_retrieved, TRJ_EINVAL,
                    "decode_device_tree: row %d has rank %d (K = %d, %d retrieval slots)", i, rank[i], K, n_retrieved);
    }
    const int32_t per_step = deepest + 1;        // a step commits at most the deepest path plus the bonus token
    TRJ_REQUIRE(n_ctx_now >= 1, TRJ_EINVAL, "decode_device_tree: empty context");
    TRJ_REQUIRE((int64_t)n_ctx_now + (int64_t)n_steps * per_step <= capacity, TRJ_ECAPACITY,
                "decode_device_tree: context buffer of %d cannot take %d steps of up to %d tokens after %d", capacity, n_steps, per_step, n_ctx_now);
    const int64_t max_len = (int64_t)n_ctx_now - 1 + (int64_t)n_steps * per_step + M;
    TRJ_REQUIRE(max_len <= c.max_seq, TRJ_ECAPACITY, "decode_device_tree: up to %lld cache rows exceed max_seq %d", (long long)max_len, c.max_seq);
    TRJ_REQUIRE(!ctx->draft_src.stream || ctx->draft_src_steps >= n_steps, TRJ_ECAPACITY,
                "decode_device_tree: the draft source covers %d steps, %d asked", ctx->draft_src_steps, n_steps);
    s = check_step_args(ctx, 1, M, M, (int32_t)max_len, 2);
    if (s != TRJ_OK) return s;
    if (n_steps == 0) return TRJ_OK;
    cudaStream_t st = (cudaStream_t)stream;
    h_off[0] = 0; h_off[1] = M;
    // the ranks travel in the staging area's token slots (the tokens themselves are built on the device)
    for (int32_t i = 0; i < M; ++i) in[i] = rank[i];
    int32_t* d_rank = ctx->loop_tree, *d_retr = d_rank + TRJ_MAX_ROWS, *d_topk = d_retr + TRJ_MAX_ROWS;
    TRJ_CHECK_CUDA(cudaMemcpyAsync(ctx->step_in, ctx->pin_in, STEP_IN_BYTES, cudaMemcpyHostToDevice, st));
    TRJ_CHECK_CUDA(cudaMemcpyAsync(d_rank, ctx->step_in, sizeof(int32_t) * M, cudaMemcpyDeviceToDevice, st));
    TRJ_CHECK_CUDA(cudaMemsetAsync(ctx->loop_state, 0, sizeof(int32_t) * 64, st));
    // the pinned staging area is shared with trj_step_host: the copy must have left it before this call returns
    TRJ_CHECK_CUDA(cudaEventRecord(ctx->order_ev, st));
    TRJ_CHECK_CUDA(cudaEventSynchronize(ctx->order_ev));
    int32_t* d_tokens = ctx->step_in, *d_parent = d_tokens + TRJ_MAX_ROWS, *d_depth = d_tokens + 2 * TRJ_MAX_ROWS;
    int32_t* d_off = d_tokens + 3 * TRJ_MAX_ROWS;
    uint64_t* d_anc = (uint64_t*)(d_tokens + STEP_IN_INTS);
    int32_t* d_pred = ctx->step_out, *d_k = d_pred + TRJ_MAX_ROWS, *d_bonus = d_k + 1, *d_path = d_k + 2;
    int32_t* d_step = ctx->loop_state, *d_overflow = ctx->loop_state + 1;
    Batch bt{seq_len, d_off, 1, M, M, (int32_t)max_len};
    auto enqueue_one = [&](cudaStream_t on) -> trj_status {
        ChainScope chain;
        LAUNCH_ON(on, PROF_ELEMENTWISE, launch_template_tokens(context, n_ctx, drafts, d_rank, M, n_retrieved, draws, d_step, d_tokens,
                                                               d_retr, on, ctx->draft_src));
        trj_status fs = forward(ctx, k_cache, v_cache, 0, bt, d_tokens, d_depth, d_anc, 2, 0, M, on);
        if (fs != TRJ_OK) return fs;
        LAUNCH_ON(on, PROF_ARGMAX, launch_topk_accept(ctx->logits, TRJ_F32, c.vocab, K, d_tokens, d_parent, d_depth, d_off, 1, M, d_topk,
                                                      d_pred, nullptr, d_k, d_path, d_bonus, true, ctx->argmax_ws, on));
        LAUNCH_ON(on, PROF_COMPACT, launch_compact(k_cache, v_cache, c.n_layers, c.max_batch, 1, kv_heads(c), c.max_seq, c.head_dim,
                                                   c.dtype, seq_len, d_k, d_path, on, ctx->compact_tickets));
        LAUNCH_ON(on, PROF_ELEMENTWISE, launch_commit_refill_tree(d_tokens, d_parent, d_depth, d_rank, d_topk, K, M, d_k, d_path, d_bonus,
                                                                  context, capacity, n_ctx, n_retrieved, draws, d_step, d_retr, drafts,
                                                                  k_log, d_overflow, on));
        return TRJ_OK;
    };
    const std::vector<uint64_t> key_of_loop = {(uint64_t)1 /* template */, (uint64_t)M, (uint64_t)K, (uint64_t)n_retrieved,
                                               (uint64_t)tree_attention_grid(1, c.n_heads, (int32_t)max_len),
                                               (uint64_t)(uintptr_t)k_cache, (uint64_t)(uintptr_t)v_cache, (uint64_t)(uintptr_t)seq_len,
                                               (uint64_t)(uintptr_t)context, (uint64_t)capacity, (uint64_t)(uintptr_t)n_ctx,
                                               (uint64_t)(uintptr_t)drafts, (uint64_t)(uintptr_t)draws, (uint64_t)(uintptr_t)k_log,
                                               (uint64_t)max_len, (uint64_t)(uintptr_t)ctx->draft_src.stream, (uint64_t)ctx->draft_src.n,
                                               (uint64_t)(uintptr_t)ctx->draft_src.take};
    return run_device_loop(ctx, key_of_loop, n_steps, enqueue_one, st);
}

