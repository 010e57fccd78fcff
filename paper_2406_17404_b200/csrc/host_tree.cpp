// Host-side integer steps around a verification step: tree layout, ancestor bitmask,
// prompt-lookup retrieval and window refill (paper Section 3.3, Appendix B, Eq. 4).
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <vector>
#include "trj_internal.h"

namespace trj {

static thread_local char g_err[512] = "";

trj_status fail(trj_status code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

trj_status tree_from_parents_impl(const int32_t* parent, int32_t M, int32_t anc_words,
                                  int32_t* depth, uint64_t* anc) {
    TRJ_REQUIRE(parent && depth && anc, TRJ_EINVAL, "tree: null pointer");
    TRJ_REQUIRE(M >= 1, TRJ_EINVAL, "tree: needs at least the root row");
    TRJ_REQUIRE(M <= TRJ_MAX_ROWS, TRJ_ECAPACITY, "tree: %d rows exceed the limit of %d", M, TRJ_MAX_ROWS);
    TRJ_REQUIRE(anc_words >= (M + 63) / 64, TRJ_ECAPACITY, "tree: anc_words %d too small for %d rows", anc_words, M);
    TRJ_REQUIRE(parent[0] == -1, TRJ_EINVAL, "tree: row 0 must be the root (parent -1)");
    std::memset(anc, 0, sizeof(uint64_t) * (size_t)M * anc_words);
    depth[0] = 0;
    anc[0] = 1ull;
    for (int32_t i = 1; i < M; ++i) {
        const int32_t p = parent[i];
        TRJ_REQUIRE(p >= 0 && p < i, TRJ_EINVAL, "tree: parent[%d] = %d is not an earlier row", i, p);
        depth[i] = depth[p] + 1;
        // a row sees what its parent sees, plus itself
        for (int32_t w = 0; w < anc_words; ++w) anc[(size_t)i * anc_words + w] = anc[(size_t)p * anc_words + w];
        anc[(size_t)i * anc_words + i / 64] |= 1ull << (i % 64);
    }
    return TRJ_OK;
}

}  // namespace trj

extern "C" const char* trj_last_error(void) { return trj::g_err; }
extern "C" const char* trj_version(void) { return "trj 0.1 (sm_100a)"; }

extern "C" trj_status trj_tree_from_parents(const int32_t* parent, int32_t M, int32_t anc_words,
                                            int32_t* depth, uint64_t* anc) {
    return trj::tree_from_parents_impl(parent, M, anc_words, depth, anc);
}

extern "C" trj_status trj_build_tree(int32_t root, const int32_t* window, int32_t W,
                                     const int32_t* branches, int32_t R, int32_t branch_len,
                                     int32_t max_rows, int32_t anc_words,
                                     int32_t* tokens, int32_t* parent, int32_t* depth,
                                     uint64_t* anc, int32_t* n_rows) {
    TRJ_REQUIRE(W >= 0 && R >= 0 && branch_len >= 0, TRJ_EINVAL, "build_tree: negative size");
    TRJ_REQUIRE(tokens && parent && depth && anc && n_rows, TRJ_EINVAL, "build_tree: null output");
    TRJ_REQUIRE(W == 0 || window, TRJ_EINVAL, "build_tree: null window");
    TRJ_REQUIRE(R * branch_len == 0 || branches, TRJ_EINVAL, "build_tree: null branches");
    TRJ_REQUIRE(max_rows <= TRJ_MAX_ROWS, TRJ_ECAPACITY, "build_tree: max_rows %d exceeds %d", max_rows, TRJ_MAX_ROWS);
    const int64_t M = 1 + (int64_t)W + (int64_t)R * branch_len;
    TRJ_REQUIRE(M <= max_rows, TRJ_ECAPACITY, "build_tree: %lld rows exceed max_rows %d", (long long)M, max_rows);
    int32_t n = 0;
    tokens[n] = root; parent[n] = -1; ++n;
    int32_t prev = 0;
    for (int32_t i = 0; i < W; ++i) { tokens[n] = window[i]; parent[n] = prev; prev = n++; }
    for (int32_t r = 0; r < R; ++r) {
        prev = 0;
        for (int32_t j = 0; j < branch_len; ++j) {
            tokens[n] = branches[(size_t)r * branch_len + j]; parent[n] = prev; prev = n++;
        }
    }
    *n_rows = n;
    return trj::tree_from_parents_impl(parent, n, anc_words, depth, anc);
}

extern "C" trj_status trj_retrieve(const int32_t* context, int32_t n, int32_t R, int32_t branch_len,
                                   const int64_t* draws, int32_t* branches) {
    TRJ_REQUIRE(n >= 1 && context, TRJ_EINVAL, "retrieve: empty context");
    TRJ_REQUIRE(R >= 0 && branch_len >= 0, TRJ_EINVAL, "retrieve: negative size");
    if (R * branch_len == 0) return TRJ_OK;
    TRJ_REQUIRE(draws && branches, TRJ_EINVAL, "retrieve: null pointer");
    std::vector<int32_t> follow;               // first index after each usable match, most recent first
    for (int32_t g = 2; g >= 1 && (int32_t)follow.size() < R; --g) {
        if (n <= g) continue;
        for (int32_t p = n - g - 1; p >= 0 && (int32_t)follow.size() < R; --p) {
            if (std::memcmp(context + p, context + n - g, sizeof(int32_t) * g) != 0) continue;
            bool seen = false;
            for (int32_t f : follow) seen |= (f == p + g);
            if (!seen) follow.push_back(p + g);
        }
    }
    for (int32_t r = 0; r < R; ++r)
        for (int32_t j = 0; j < branch_len; ++j) {
            const size_t slot = (size_t)r * branch_len + j;
            if (r < (int32_t)follow.size() && follow[r] + j < n) {
                branches[slot] = context[follow[r] + j];
            } else {
                TRJ_REQUIRE(draws[slot] >= 0, TRJ_EINVAL, "retrieve: negative random draw");
                branches[slot] = context[draws[slot] % n];
            }
        }
    return TRJ_OK;
}

extern "C" trj_status trj_refill_window(const int32_t* parent, const int32_t* node_argmax, int32_t M,
                                        int32_t best, int32_t W, const int32_t* context, int32_t n,
                                        const int64_t* draws, int32_t* window) {
    TRJ_REQUIRE(parent && node_argmax && M >= 1, TRJ_EINVAL, "refill: null tree");
    TRJ_REQUIRE(best >= 0 && best < M, TRJ_EINVAL, "refill: winner %d outside the tree", best);
    TRJ_REQUIRE(W >= 0 && (W == 0 || (window && draws && context && n >= 1)), TRJ_EINVAL, "refill: null pointer");
    int32_t filled = 0, cur = best;
    while (filled < W) {
        int32_t child = -1;
        for (int32_t c = cur + 1; c < M; ++c)
            if (parent[c] == cur) { child = c; break; }
        if (child < 0) break;
        window[filled++] = node_argmax[child];
        cur = child;
    }
    for (; filled < W; ++filled) {
        TRJ_REQUIRE(draws[filled] >= 0, TRJ_EINVAL, "refill: negative random draw");
        window[filled] = context[draws[filled] % n];
    }
    return TRJ_OK;
}

extern "C" trj_status trj_refill_tree(const int32_t* parent, const int32_t* rank, int32_t M, const int32_t* topk, int32_t K,
                                      int32_t best, const int32_t* context, int32_t n, const int64_t* draws,
                                      const int32_t* retrieved, int32_t n_retrieved, int32_t* tokens) {
    TRJ_REQUIRE(parent && rank && topk && M >= 1, TRJ_EINVAL, "refill_tree: null tree");
    TRJ_REQUIRE(M <= TRJ_MAX_ROWS, TRJ_ECAPACITY, "refill_tree: %d rows exceed the limit of %d", M, TRJ_MAX_ROWS);
    TRJ_REQUIRE(K >= 1 && K <= TRJ_MAX_TOPK, TRJ_EINVAL, "refill_tree: K = %d outside 1..%d", K, TRJ_MAX_TOPK);
    TRJ_REQUIRE(best >= 0 && best < M, TRJ_EINVAL, "refill_tree: winner %d outside the tree", best);
    TRJ_REQUIRE(M == 1 || (tokens && draws && context && n >= 1), TRJ_EINVAL, "refill_tree: null pointer");
    TRJ_REQUIRE(n_retrieved >= 0 && (n_retrieved == 0 || retrieved), TRJ_EINVAL, "refill_tree: null retrieved tokens");
    // depth of every row, and the rows below the winner along its own path (lowest-index child at every level)
    int32_t depth[TRJ_MAX_ROWS], below[TRJ_MAX_ROWS];
    depth[0] = 0;
    for (int32_t i = 1; i < M; ++i) {
        TRJ_REQUIRE(parent[i] >= 0 && parent[i] < i, TRJ_EINVAL, "refill_tree: parent[%d] = %d is not an earlier row", i, parent[i]);
        depth[i] = depth[parent[i]] + 1;
    }
    int32_t n_below = 0;
    for (int32_t cur = best;;) {
        int32_t child = -1;
        for (int32_t c = cur + 1; c < M; ++c)
            if (parent[c] == cur) { child = c; break; }
        if (child < 0) break;
        below[n_below++] = child;
        cur = child;
    }
    for (int32_t i = 1; i < M; ++i) {
        const int32_t r = rank[i];
        if (r < 0) {
            TRJ_REQUIRE(-1 - r < n_retrieved, TRJ_EINVAL, "refill_tree: row %d wants retrieval slot %d of %d", i, -1 - r, n_retrieved);
            tokens[i - 1] = retrieved[-1 - r];
        } else if (depth[i] <= n_below) {
            TRJ_REQUIRE(r < K, TRJ_EINVAL, "refill_tree: row %d has rank %d but K = %d", i, r, K);
            tokens[i - 1] = topk[(size_t)below[depth[i] - 1] * K + r];
        } else {
            TRJ_REQUIRE(draws[i - 1] >= 0, TRJ_EINVAL, "refill_tree: negative random draw");
            tokens[i - 1] = context[draws[i - 1] % n];
        }
    }
    return TRJ_OK;
}
