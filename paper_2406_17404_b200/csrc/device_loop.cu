// Device-side drafting and refill: the integer bookkeeping between two verification steps (prompt-lookup
// retrieval, tree tokens, commit of the accepted tokens, next Jacobi window), so that a decode loop needs no
// host round trip per step.  Each kernel is one warp; the work is a few hundred integer operations.
// Semantics are those of the host functions trj_retrieve / trj_build_tree / trj_refill_window (Section 3.3:
// retrieval from the tokens seen so far, refill from the chosen path's own predictions; Eq. 4: ahead noise).
#include <cstdint>
#include "trj_internal.h"

namespace trj {
namespace {

constexpr int MAX_BRANCHES = 64;          // R is bounded by the tree size (R * Lr < TRJ_MAX_ROWS)

// Prompt-lookup matches, by a whole warp: the positions that followed the R most recent earlier occurrences of the
// context's last two tokens, then of its last token (no position twice).  Every lane ends up with the same list.
// The context is walked from its end in blocks of FOLLOW_BLOCK tokens that the warp first copies to shared memory
// (32 independent loads per lane, one trip to L2 per block instead of one per 32 tokens).
constexpr int FOLLOW_BLOCK = 1024;
__device__ __forceinline__ int find_follows(const int32_t* __restrict__ context, int n, int R, int* follow, int lane) {
    __shared__ int32_t blk[FOLLOW_BLOCK + 1];                // tokens lo .. lo + FOLLOW_BLOCK (one more: the pair's second token)
    int nf = 0;
    for (int g = 2; g >= 1 && nf < R; --g) {
        if (n <= g) continue;
        const int t0 = context[n - g], t1 = context[n - 1];          // g == 1: t0 == t1
        // candidate positions p = n - g - 1 down to 0
        for (int hi = n - g - 1; hi >= 0 && nf < R; hi -= FOLLOW_BLOCK) {
            const int lo = max(hi - FOLLOW_BLOCK + 1, 0);
            __syncwarp();
            for (int i = lo + lane; i <= hi + 1; i += 32) blk[i - lo] = context[i];      // hi + 1 <= n - g < n
            __syncwarp();
            for (int base = hi; base >= lo && nf < R; base -= 32) {
                const int p = base - lane;
                bool match = false;
                if (p >= lo) match = blk[p - lo] == t0 && (g == 1 || blk[p - lo + 1] == t1);
                unsigned m = __ballot_sync(0xffffffffu, match);
                while (m && nf < R) {                        // lane 0 holds the largest p: ascending lanes = descending p
                    const int l = __ffs(m) - 1;
                    m &= m - 1;
                    const int f = base - l + g;
                    bool seen = false;
                    for (int i = 0; i < nf; ++i) seen |= follow[i] == f;
                    if (!seen) follow[nf++] = f;
                }
            }
        }
    }
    return nf;
}

// tokens[0] = root (last committed token), tokens[1..W] = window, then R branches of Lr tokens: for each of the R
// most recent earlier occurrences of the context's last two tokens (then of its last token), the Lr tokens that
// followed; missing slots are ahead noise, context[draw % n].  `step` (may be null) selects this step's draws.
// An external draft source (may be absent) overrides the start of branch 0: src.stream[i] is its guess for the token
// at context position i, and step s takes src.take[s] of them, from position n on.
__global__ void __launch_bounds__(32) draft_tokens_kernel(const int32_t* __restrict__ context, const int32_t* __restrict__ n_ctx,
                                                          const int32_t* __restrict__ window, int W, int R, int Lr,
                                                          const int64_t* __restrict__ draws, const int32_t* __restrict__ step,
                                                          int32_t* __restrict__ tokens, const DraftSource src) {
    pdl_prologue();
    const int lane = threadIdx.x;
    const int n = *n_ctx;
    const int64_t* my_draws = draws + (step ? (size_t)*step * (size_t)(W + R * Lr) : 0);
    if (lane == 0) tokens[0] = context[n - 1];
    for (int i = lane; i < W; i += 32) tokens[1 + i] = window[i];
    // every lane keeps the same list of follow positions (first index after a match), most recent match first
    int follow[MAX_BRANCHES];
    const int nf = find_follows(context, n, R, follow, lane);
    for (int slot = lane; slot < R * Lr; slot += 32) {
        const int r = slot / Lr, j = slot % Lr;
        int32_t tok;
        if (r < nf && follow[r] + j < n) tok = context[follow[r] + j];
        else tok = context[(uint64_t)my_draws[W + slot] % (uint64_t)n];
        if (src.stream && r == 0 && j < src.take[step ? *step : 0] && n + j < src.n) tok = src.stream[n + j];
        tokens[1 + W + slot] = tok;
    }
}

// Appends the accepted draft tokens and the bonus token to the context, refills the window from the predictions
// below the winning node (lowest-index child at every level, then ahead noise on the grown context), and advances
// the step counter.  A context that would overflow `capacity` is left untouched and flagged in *overflow.
__global__ void __launch_bounds__(32) commit_refill_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                                                           const int32_t* __restrict__ node_argmax, int M,
                                                           const int32_t* __restrict__ k_acc, const int32_t* __restrict__ path,
                                                           const int32_t* __restrict__ bonus, int32_t* __restrict__ context,
                                                           int capacity, int32_t* __restrict__ n_ctx, int W, int draws_per_step,
                                                           const int64_t* __restrict__ draws, int32_t* __restrict__ step,
                                                           int32_t* __restrict__ window, int32_t* __restrict__ k_log,
                                                           int32_t* __restrict__ overflow) {
    pdl_prologue();
    const int lane = threadIdx.x;
    const int n = *n_ctx, k = *k_acc;
    const int s = step ? *step : 0;
    const int64_t* my_draws = draws + (size_t)s * (size_t)draws_per_step;
    if (n + k + 1 > capacity) {
        if (lane == 0 && overflow) *overflow = 1;
        return;
    }
    for (int j = lane; j < k; j += 32) context[n + j] = tokens[path[j + 1]];
    if (lane == 0) context[n + k] = *bonus;
    __syncwarp();
    if (lane == 0) {
        const int n_new = n + k + 1;
        int filled = 0, cur = path[k];
        while (filled < W) {
            int child = -1;
            for (int c = cur + 1; c < M; ++c)
                if (parent[c] == cur) { child = c; break; }
            if (child < 0) break;
            window[filled++] = node_argmax[child];
            cur = child;
        }
        for (; filled < W; ++filled) window[filled] = context[(uint64_t)my_draws[filled] % (uint64_t)n_new];
        *n_ctx = n_new;
        if (k_log) k_log[s] = k;
        if (step) *step = s + 1;
    }
}

// ---- static tree templates with top-K siblings (Appendix B) ----
// The step's tree tokens: the root, the drafts the previous step's refill left, and the retrieval path (rows of rank
// -1-j) refreshed from the current context: slot j takes the j-th token after the most recent earlier occurrence of
// the context's last two tokens (then of its last token), or ahead noise context[draw % n] (Eq. 4).  The retrieved
// tokens are kept in `retr` for the refill.  draws of step s: [0, M-1) refill, [M-1, M-1+n_retr) retrieval.
__global__ void __launch_bounds__(32) template_tokens_kernel(const int32_t* __restrict__ context, const int32_t* __restrict__ n_ctx,
                                                             const int32_t* __restrict__ drafts, const int32_t* __restrict__ rank,
                                                             int M, int n_retr, const int64_t* __restrict__ draws,
                                                             const int32_t* __restrict__ step, int32_t* __restrict__ tokens,
                                                             int32_t* __restrict__ retr, const DraftSource src) {
    pdl_prologue();
    const int lane = threadIdx.x;
    const int n = *n_ctx;
    const int64_t* my_draws = draws + (size_t)*step * (size_t)(M - 1 + n_retr);
    int follow[1];
    const int nf = n_retr > 0 ? find_follows(context, n, 1, follow, lane) : 0;
    for (int j = lane; j < n_retr; j += 32) {
        int32_t tok = (nf > 0 && follow[0] + j < n) ? context[follow[0] + j] : context[(uint64_t)my_draws[M - 1 + j] % (uint64_t)n];
        // an external draft source (may be absent) overrides the start of the retrieval path, as it does for branch 0
        if (src.stream && j < src.take[*step] && n + j < src.n) tok = src.stream[n + j];
        retr[j] = tok;
    }
    __syncwarp();
    if (lane == 0) tokens[0] = context[n - 1];
    for (int i = 1 + lane; i < M; i += 32) tokens[i] = rank[i] < 0 ? retr[-1 - rank[i]] : drafts[i - 1];
}

// After a step over a template: appends the accepted draft tokens and the bonus token to the context and writes the
// next step's drafts.  Candidates for depth d come from the d-th row below the winner along its own path
// (lowest-index child at every level): row i of depth d and rank r takes topk[that row][r]; depths the path does not
// reach are ahead noise on the grown context; retrieval rows take this step's retrieved tokens.
__global__ void __launch_bounds__(32) commit_refill_tree_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                                                                const int32_t* __restrict__ depth, const int32_t* __restrict__ rank,
                                                                const int32_t* __restrict__ topk, int K, int M,
                                                                const int32_t* __restrict__ k_acc, const int32_t* __restrict__ path,
                                                                const int32_t* __restrict__ bonus, int32_t* __restrict__ context,
                                                                int capacity, int32_t* __restrict__ n_ctx, int n_retr,
                                                                const int64_t* __restrict__ draws, int32_t* __restrict__ step,
                                                                const int32_t* __restrict__ retr, int32_t* __restrict__ drafts,
                                                                int32_t* __restrict__ k_log, int32_t* __restrict__ overflow) {
    pdl_prologue();
    __shared__ int32_t below[TRJ_MAX_ROWS];
    __shared__ int n_below_s;
    const int lane = threadIdx.x;
    const int n = *n_ctx, k = *k_acc;
    const int s = *step;
    const int64_t* my_draws = draws + (size_t)s * (size_t)(M - 1 + n_retr);
    if (n + k + 1 > capacity) {
        if (lane == 0 && overflow) *overflow = 1;
        return;
    }
    for (int j = lane; j < k; j += 32) context[n + j] = tokens[path[j + 1]];
    if (lane == 0) context[n + k] = *bonus;
    // the rows below the winner along its own path: the lowest-index child at every level, found by the whole warp
    // over a copy of the parent array in shared memory
    __shared__ int32_t par_s[TRJ_MAX_ROWS];
    for (int i = lane; i < M; i += 32) par_s[i] = parent[i];
    __syncwarp();
    int nb = 0;
    for (int cur = path[k];;) {
        int child = -1;
        for (int c0 = cur + 1; c0 < M && child < 0; c0 += 32) {
            const int c = c0 + lane;
            const unsigned hit = __ballot_sync(0xffffffffu, c < M && par_s[c] == cur);
            if (hit) child = c0 + __ffs(hit) - 1;
        }
        if (child < 0) break;
        if (lane == 0) below[nb] = child;
        ++nb;
        cur = child;
    }
    if (lane == 0) n_below_s = nb;
    __syncwarp();
    const int n_new = n + k + 1, n_below = n_below_s;
    for (int i = 1 + lane; i < M; i += 32) {
        const int r = rank[i];
        int32_t tok;
        if (r < 0) tok = retr[-1 - r];
        else if (depth[i] <= n_below) tok = topk[(size_t)below[depth[i] - 1] * K + r];
        else tok = context[(uint64_t)my_draws[i - 1] % (uint64_t)n_new];
        drafts[i - 1] = tok;
    }
    __syncwarp();
    if (lane == 0) {
        *n_ctx = n_new;
        if (k_log) k_log[s] = k;
        *step = s + 1;
    }
}

}  // namespace

cudaError_t launch_template_tokens(const int32_t* context, const int32_t* n_ctx, const int32_t* drafts, const int32_t* rank,
                                   int32_t M, int32_t n_retr, const int64_t* draws, const int32_t* step, int32_t* tokens,
                                   int32_t* retr, cudaStream_t st, const DraftSource& src) {
    count_launch();
    cudaError_t e = launch_chain(template_tokens_kernel, dim3(1), dim3(32), 0, st, context, n_ctx, drafts, rank, M, n_retr, draws, step,
                                 tokens, retr, src);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_commit_refill_tree(const int32_t* tokens, const int32_t* parent, const int32_t* depth, const int32_t* rank,
                                      const int32_t* topk, int32_t K, int32_t M, const int32_t* k_acc, const int32_t* path,
                                      const int32_t* bonus, int32_t* context, int32_t capacity, int32_t* n_ctx, int32_t n_retr,
                                      const int64_t* draws, int32_t* step, const int32_t* retr, int32_t* drafts, int32_t* k_log,
                                      int32_t* overflow, cudaStream_t st) {
    count_launch();
    cudaError_t e = launch_chain(commit_refill_tree_kernel, dim3(1), dim3(32), 0, st, tokens, parent, depth, rank, topk, K, M, k_acc,
                                 path, bonus, context, capacity, n_ctx, n_retr, draws, step, retr, drafts, k_log, overflow);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_draft_tokens(const int32_t* context, const int32_t* n_ctx, const int32_t* window, int32_t W, int32_t R,
                                int32_t Lr, const int64_t* draws, const int32_t* step, int32_t* tokens, cudaStream_t st,
                                const DraftSource& src) {
    if (R > MAX_BRANCHES) return cudaErrorInvalidValue;
    count_launch();
    cudaError_t e = launch_chain(draft_tokens_kernel, dim3(1), dim3(32), 0, st, context, n_ctx, window, W, R, Lr, draws, step, tokens, src);
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_commit_refill(const int32_t* tokens, const int32_t* parent, const int32_t* node_argmax, int32_t M,
                                 const int32_t* k_acc, const int32_t* path, const int32_t* bonus, int32_t* context,
                                 int32_t capacity, int32_t* n_ctx, int32_t W, int32_t draws_per_step, const int64_t* draws,
                                 int32_t* step, int32_t* window, int32_t* k_log, int32_t* overflow, cudaStream_t st) {
    count_launch();
    cudaError_t e = launch_chain(commit_refill_kernel, dim3(1), dim3(32), 0, st, tokens, parent, node_argmax, M, k_acc, path, bonus,
                                 context, capacity, n_ctx, W, draws_per_step, draws, step, window, k_log, overflow);
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace trj
