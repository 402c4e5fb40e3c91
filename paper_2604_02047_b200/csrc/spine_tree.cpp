// Host side of Goose's decoding loop: BuildSpineTree (Algorithm 1), ContextMatch (the n-gram lookup
// described after Algorithm 2) and the spine-ratio tiers / EMA of the hyper-parameter table.
// Plain host C++ behind the C ABI: every pointer here is a HOST pointer.  Tree construction is <1% of the
// loop's wall clock in the paper and stays on the CPU; it emits parent[] / draft_tok[] in the
// topological, spine-first order the verification kernels expect.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

#include "goose.h"

namespace {

struct Tree {
    int32_t* tok;
    int32_t* parent;
    uint8_t* is_spine;
    std::vector<int> depth;   // nodes from the fork (0 on the spine)
    int n = 0;
    int cap;

    bool child_has(int p, int32_t t) const {
        for (int c = p + 1; c < n; ++c)
            if (parent[c] == p && tok[c] == t) return true;
        return false;
    }
    int add(int p, int32_t t, bool spine, int dep) {
        tok[n] = t; parent[n] = p; if (is_spine) is_spine[n] = spine ? 1 : 0;
        depth.push_back(dep);
        return n++;
    }
};

}  // namespace

extern "C" {

int goose_build_spine_tree(int32_t anchor, const int32_t* chain, int m, const int32_t* adj_ids, int table_rows, int K,
                           int B, int D, float r, float rho, int32_t* draft_tok, int32_t* parent, uint8_t* is_spine,
                           int32_t* n_nodes, int32_t* n_spine) {
    if (!draft_tok || !parent || !n_nodes || m < 0 || (m > 0 && !chain) || B < 1 || B > GOOSE_MAX_B || D < 1 ||
        K < 0 || table_rows < 0 || (K > 0 && table_rows > 0 && !adj_ids) || !(r > 0.f && r < 1.f) ||
        !(rho > 0.f && rho < 1.f))
        return GOOSE_EINVAL;
    // budget split (Algorithm 1, lines 1-3); double arithmetic so that floor(B*r) is the paper's value
    const int b_s = std::min(m, (int)std::floor((double)B * (double)r));
    const int b_r = (int)std::floor((double)(B - 1 - b_s) * (1.0 - (double)rho));
    const int b_rho = B - 1 - b_s - b_r;

    Tree t{draft_tok, parent, is_spine, {}, 0, B};
    t.add(-1, anchor, true, 0);
    for (int i = 1; i <= b_s; ++i) t.add(i - 1, chain[i - 1], true, 0);       // step 1: node i is spine node d_i

    std::vector<int> branch;
    auto attach = [&](int node, int count) {                                   // ranked, duplicate-free successors
        const int32_t tk = t.tok[node];
        if (tk < 0 || tk >= table_rows) return;
        int got = 0;
        for (int j = 0; j < K && got < count && t.n < B; ++j) {
            const int32_t s = adj_ids[(size_t)tk * K + j];
            if (s < 0 || t.child_has(node, s)) continue;
            branch.push_back(t.add(node, s, false, 1));
            ++got;
        }
    };
    attach(0, b_r);                                                            // step 2: root branches
    double H = 0.0;
    for (int j = 1; j <= b_s; ++j) H += 1.0 / j;
    for (int i = 1; i <= b_s; ++i)                                             // step 3: harmonic spine branches
        attach(i, (int)std::floor((double)b_rho * (1.0 / i) / H));
    // step 4: breadth-first extension of the branch leaves, one top successor each, up to D nodes per branch
    std::vector<int> frontier = branch, next;
    while (!frontier.empty() && t.n < B) {
        next.clear();
        for (int leaf : frontier) {
            if (t.n >= B) break;
            if (t.depth[leaf] >= D) continue;
            const int32_t tk = t.tok[leaf];
            if (tk < 0 || tk >= table_rows) continue;
            for (int j = 0; j < K; ++j) {
                const int32_t s = adj_ids[(size_t)tk * K + j];
                if (s < 0 || t.child_has(leaf, s)) continue;
                next.push_back(t.add(leaf, s, false, t.depth[leaf] + 1));
                break;
            }
        }
        frontier.swap(next);
    }
    *n_nodes = t.n;
    if (n_spine) *n_spine = b_s + 1;
    return GOOSE_OK;
}

int goose_pad_tree(int32_t* draft_tok, int32_t* parent, int n_nodes, int B) {
    if (!draft_tok || !parent || n_nodes < 1 || n_nodes > B) return GOOSE_EINVAL;
    // padding nodes hang on the root with negative tokens: no argmax can equal them, so they are never accepted
    for (int i = n_nodes; i < B; ++i) { parent[i] = 0; draft_tok[i] = -1 - i; }
    return GOOSE_OK;
}

int goose_context_match(const int32_t* ctx, int n_ctx, int max_len, int32_t* chain, int32_t* chain_len,
                        int32_t* consensus) {
    if (!ctx || n_ctx < 0 || max_len < 0 || !chain_len || (max_len > 0 && !chain)) return GOOSE_EINVAL;
    static const int kN[3] = {5, 4, 3};
    int found_n = 0, found_p = -1;
    int32_t firsts[3];
    int n_first = 0;
    for (int q = 0; q < 3; ++q) {
        const int n = kN[q];
        if (n_ctx <= n) continue;
        const int32_t* query = ctx + n_ctx - n;
        for (int p = n_ctx - n - 1; p >= 0; --p) {                              // most recent earlier occurrence
            if (std::equal(query, query + n, ctx + p)) {
                if (!found_n) { found_n = n; found_p = p; }
                if (max_len > 0) firsts[n_first++] = ctx[p + n];
                break;
            }
        }
    }
    int len = 0;
    if (found_n) {
        const int start = found_p + found_n;
        len = std::min(max_len, n_ctx - start);
        for (int i = 0; i < len; ++i) chain[i] = ctx[start + i];
    }
    *chain_len = len;
    bool agree = false;
    for (int a = 0; a < n_first; ++a)
        for (int b = a + 1; b < n_first; ++b) agree |= (firsts[a] == firsts[b]);
    if (consensus) *consensus = agree ? 1 : 0;
    return GOOSE_OK;
}

float goose_spine_ratio_tier(float p_hat) { return p_hat < 0.2f ? 0.15f : (p_hat < 0.4f ? 0.30f : 0.50f); }

float goose_spine_ema(float p_hat, int accepted_spine, int drafted_spine) {
    if (drafted_spine <= 0) return p_hat;
    return 0.7f * p_hat + 0.3f * ((float)accepted_spine / (float)drafted_spine);
}

}  // extern "C"
