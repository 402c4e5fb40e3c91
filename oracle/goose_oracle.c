/*
 * CPU oracle for the Goose tree-verification step.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64, written from the paper's definitions; it shares no code, header,
 * table or helper with the CUDA library and must never be called from the product path
 * (only the tests, the smoke check and the benchmark's CPU-baseline leg use it).
 *
 * Every function below is the plain definition of what the step computes:
 *   - tree attention:  the "tree attention mask ... lets each node attend only to its
 *     root-to-node ancestors" (Sec. 4, Stage 1; Algorithm 1 "Ensure"; Algorithm 3 step 1),
 *     i.e. softmax(scale * q.K^T + mask) V with mask = prefix + ancestors (self included).
 *   - node top-k:      per-node greedy argmax (Algorithm 3 step 2) and the batched top-K
 *     harvested from every row of the forward's logits (App. "Aggressive logit harvesting").
 *   - accept:          UnifiedGreedyWalk (Algorithm 3), literal pointer walk.
 *   - kv compaction:   the paper never describes it; the reading used here is "keep the
 *     accepted nodes' K/V rows, in path order, directly after the prefix".
 *
 * Per-sequence node counts (the paper's batched prototype pads finished requests and pays for them, App.
 * "Batch-Size Sweep"; its Discussion leaves a production batched path open): every function that takes a tree takes
 * an optional n_nodes[S] (NULL = B nodes everywhere).  Nodes i >= n_nodes[s] do not exist: nothing of theirs is read
 * (parent, token, query, K/V row, logits row may hold anything) and nothing is written for them; the result for the
 * nodes that exist is BY DEFINITION the result on the tree cut to its first n_nodes[s] nodes (a tree in topological
 * order stays a tree when cut), and n_nodes[s] = 0 is a sequence that has left the batch: no reads, no moves,
 * accept_len 0, bonus -1, path all -1, new_ctx = ctx.  Pinned against this file's own B-node functions on explicitly
 * cut inputs.
 *
 * bf16 inputs arrive as uint16 bit patterns; bf16 -> double is exact.
 * No blocking, no fusion, no reordering: one output element at a time.
 * All functions are pinned by tests that do not depend on this file's own formulas.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* nodes of sequence s: n_nodes[s] when given (it must lie in [0, B]), else B; -1 = invalid */
static int nodes_of(const int32_t* n_nodes, int s, int B) {
    if (!n_nodes) return B;
    return (n_nodes[s] < 0 || n_nodes[s] > B) ? -1 : n_nodes[s];
}

/* ------------------------------------------------------------------ ancestors
 * A(0) = {0};  A(i) = A(parent[i]) U {i}   (root-to-node path, node included).
 * vis[j] = 1 iff j in A(i).  Returns 0, or -1 if parent[] is not a rooted tree in
 * topological order (parent[0] = -1, 0 <= parent[i] < i). */
static int ancestors_of(const int32_t* parent, int B, int i, unsigned char* vis) {
    memset(vis, 0, (size_t)B);
    int v = i;
    int steps = 0;
    while (v != -1) {
        if (v < 0 || v >= B || steps > B) return -1;
        vis[v] = 1;
        int p = parent[v];
        if (v == 0) {
            if (p != -1) return -1;
        } else if (p < 0 || p >= v) {
            return -1;
        }
        v = p;
        ++steps;
    }
    return vis[0] ? 0 : -1;
}

/* The ancestor set of node i as the tests see it: vis[j] = 1 iff j in A(i), j = 0..B-1.  Same return codes. */
int oracle_ancestors(const int32_t* parent, int B, int i, unsigned char* vis) {
    if (B < 1 || i < 0 || i >= B) return -1;
    return ancestors_of(parent, B, i, vis);
}

int oracle_check_parent(const int32_t* parent, int B) {
    if (B < 1 || parent[0] != -1) return -1;
    for (int i = 1; i < B; ++i)
        if (parent[i] < 0 || parent[i] >= i) return -1;
    return 0;
}

/* ------------------------------------------------------------------ tree attention, one row
 * Node i of sequence s, query head h.  Visible keys: prefix rows 0..ctx-1 and tree rows ctx+j, j in A(i).
 *   s_j = scale * sum_d q[d] K[j][d];  p_j = exp(s_j - max) / sum exp(s - max);  out = sum_j p_j V[j].
 * K/V layout: [row][Hkv][D], sequence s owns rows row_off[s] .. row_off[s]+ctx+B-1.
 * Grouped-query attention (the 8B models of the paper's evaluation, Sec. 5 set-up, have 32 query heads over 8
 * key/value heads): the H query heads are split into Hkv groups of H/Hkv consecutive heads, and every head of a
 * group reads key/value head hk = h / (H/Hkv).  Hkv == H is ordinary multi-head attention (hk = h). */
static int attn_row(const uint16_t* q, const uint16_t* kc, const uint16_t* vc, int64_t row0, int ctx,
                    const int32_t* parent, int B /* nodes of this sequence's tree */, int H, int Hkv, int D, double scale, int i, int h,
                    const uint16_t* qrow /* q[s][i][h][:] */, double* out /* [D] */, double* lse) {
    (void)q;
    if (Hkv < 1 || H % Hkv != 0) return -3;
    const int hk = h / (H / Hkv);
    int n = ctx + B;
    unsigned char* vis = (unsigned char*)malloc((size_t)B);
    double* sc = (double*)malloc(sizeof(double) * (size_t)n);
    if (!vis || !sc) { free(vis); free(sc); return -2; }
    if (ancestors_of(parent, B, i, vis) != 0) { free(vis); free(sc); return -1; }

    double mx = -INFINITY;
    for (int j = 0; j < n; ++j) {
        int visible = (j < ctx) ? 1 : vis[j - ctx];
        if (!visible) { sc[j] = -INFINITY; continue; }
        const uint16_t* krow = kc + ((size_t)(row0 + j) * Hkv + hk) * D;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += bf16_to_f64(qrow[d]) * bf16_to_f64(krow[d]);
        sc[j] = scale * acc;
        if (sc[j] > mx) mx = sc[j];
    }
    double denom = 0.0;
    for (int j = 0; j < n; ++j)
        if (sc[j] != -INFINITY) denom += exp(sc[j] - mx);
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    for (int j = 0; j < n; ++j) {
        if (sc[j] == -INFINITY) continue;
        double p = exp(sc[j] - mx) / denom;
        const uint16_t* vrow = vc + ((size_t)(row0 + j) * Hkv + hk) * D;
        for (int d = 0; d < D; ++d) out[d] += p * bf16_to_f64(vrow[d]);
    }
    if (lse) *lse = mx + log(denom);
    free(vis);
    free(sc);
    return 0;
}

/* Full output: out fp64 [S][B][H][D], lse fp64 [S][B][H] (may be NULL). Returns 0 or <0.
 * q has H heads, the caches Hkv heads (H a multiple of Hkv).  n_nodes [S] or NULL: rows of nodes that do not exist are
 * left untouched. */
int oracle_tree_attn_n(const uint16_t* q, const uint16_t* kc, const uint16_t* vc, const int64_t* row_off,
                       const int32_t* ctx_len, const int32_t* parent, const int32_t* n_nodes, int S, int B, int H, int Hkv,
                       int D, double scale, double* out, double* lse) {
    int rc = 0;
    long total = (long)S * B * H;
    for (int s = 0; s < S; ++s)
        if (nodes_of(n_nodes, s, B) < 0) return -4;
#pragma omp parallel for schedule(dynamic, 4)
    for (long t = 0; t < total; ++t) {
        int h = (int)(t % H);
        int i = (int)((t / H) % B);
        int s = (int)(t / ((long)H * B));
        const int n = nodes_of(n_nodes, s, B);
        if (i >= n) continue;                              /* the node does not exist */
        const uint16_t* qrow = q + (((size_t)s * B + i) * H + h) * D;
        int r = attn_row(q, kc, vc, row_off[s], ctx_len[s], parent + (size_t)s * B, n, H, Hkv, D, scale, i, h, qrow,
                         out + (size_t)t * D, lse ? lse + t : NULL);
        if (r != 0) {
#pragma omp critical
            rc = r;
        }
    }
    return rc;
}

int oracle_tree_attn_gqa(const uint16_t* q, const uint16_t* kc, const uint16_t* vc, const int64_t* row_off,
                         const int32_t* ctx_len, const int32_t* parent, int S, int B, int H, int Hkv, int D,
                         double scale, double* out, double* lse) {
    return oracle_tree_attn_n(q, kc, vc, row_off, ctx_len, parent, NULL, S, B, H, Hkv, D, scale, out, lse);
}

int oracle_tree_attn(const uint16_t* q, const uint16_t* kc, const uint16_t* vc, const int64_t* row_off,
                     const int32_t* ctx_len, const int32_t* parent, int S, int B, int H, int D,
                     double scale, double* out, double* lse) {
    return oracle_tree_attn_gqa(q, kc, vc, row_off, ctx_len, parent, S, B, H, H, D, scale, out, lse);
}

/* Sampled rows: for each sample n the row (s,i,h) = (ss[n], si[n], sh[n]); out [n][D], lse [n]. */
int oracle_tree_attn_rows_gqa(const uint16_t* q, const uint16_t* kc, const uint16_t* vc, const int64_t* row_off,
                              const int32_t* ctx_len, const int32_t* parent, int S, int B, int H, int Hkv, int D,
                              double scale, int n_samples, const int32_t* ss, const int32_t* si,
                              const int32_t* sh, double* out, double* lse) {
    int rc = 0;
    (void)S;
#pragma omp parallel for schedule(dynamic, 1)
    for (int n = 0; n < n_samples; ++n) {
        int s = ss[n], i = si[n], h = sh[n];
        const uint16_t* qrow = q + (((size_t)s * B + i) * H + h) * D;
        int r = attn_row(q, kc, vc, row_off[s], ctx_len[s], parent + (size_t)s * B, B, H, Hkv, D, scale, i, h, qrow,
                         out + (size_t)n * D, lse ? lse + n : NULL);
        if (r != 0) {
#pragma omp critical
            rc = r;
        }
    }
    return rc;
}

int oracle_tree_attn_rows(const uint16_t* q, const uint16_t* kc, const uint16_t* vc, const int64_t* row_off,
                          const int32_t* ctx_len, const int32_t* parent, int S, int B, int H, int D,
                          double scale, int n_samples, const int32_t* ss, const int32_t* si,
                          const int32_t* sh, double* out, double* lse) {
    return oracle_tree_attn_rows_gqa(q, kc, vc, row_off, ctx_len, parent, S, B, H, H, D, scale, n_samples, ss, si, sh,
                                     out, lse);
}

/* ------------------------------------------------------------------ per-node argmax + top-k
 * Order the indices of a row by (value descending, index ascending), values compared as real
 * numbers (so -0.0 == +0.0); the first k are the top-k, the first one is the greedy argmax. */
typedef struct { double v; int32_t idx; } vi_t;

static int cmp_vi(const void* a, const void* b) {
    const vi_t* x = (const vi_t*)a;
    const vi_t* y = (const vi_t*)b;
    if (x->v > y->v) return -1;
    if (x->v < y->v) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

/* n_nodes [rows / B] or NULL: row r = s * B + i belongs to node i of sequence s; rows of nodes that do not exist are
 * neither read nor written. */
int oracle_node_topk_n(const uint16_t* logits, int rows, int V, int64_t ldl, int k, const int32_t* n_nodes, int B,
                       int32_t* argmax, int32_t* topk_ids, double* topk_vals) {
    if (k < 1 || k > V) return -1;
    if (n_nodes && (B < 1 || rows % B != 0)) return -1;
    if (n_nodes)
        for (int s = 0; s < rows / B; ++s)
            if (nodes_of(n_nodes, s, B) < 0) return -4;
    int rc = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < rows; ++r) {
        if (n_nodes && r % B >= n_nodes[r / B]) continue;
        vi_t* a = (vi_t*)malloc(sizeof(vi_t) * (size_t)V);
        if (!a) {
#pragma omp critical
            rc = -2;
            continue;
        }
        for (int j = 0; j < V; ++j) {
            a[j].v = bf16_to_f64(logits[(size_t)r * ldl + j]);
            a[j].idx = j;
        }
        qsort(a, (size_t)V, sizeof(vi_t), cmp_vi);   /* full sort; (value, index) is a total order */
        argmax[r] = a[0].idx;
        for (int j = 0; j < k; ++j) {
            topk_ids[(size_t)r * k + j] = a[j].idx;
            if (topk_vals) topk_vals[(size_t)r * k + j] = a[j].v;
        }
        free(a);
    }
    return rc;
}

int oracle_node_topk(const uint16_t* logits, int rows, int V, int64_t ldl, int k,
                     int32_t* argmax, int32_t* topk_ids, double* topk_vals) {
    return oracle_node_topk_n(logits, rows, V, ldl, k, NULL, 0, argmax, topk_ids, topk_vals);
}

/* ------------------------------------------------------------------ UnifiedGreedyWalk (Algorithm 3)
 * v <- root; while v has children: if a spine-tagged child's token equals argmax[v] take it;
 * else if a branch-tagged child's token equals argmax[v] take it; else stop.  bonus = argmax[v].
 * tag == NULL: no source tags; the matching child with the lowest index is taken (with distinct
 * sibling tokens at most one child can match, so the priority never changes the path).
 * path [S][B]: path[0] = 0, then the accepted nodes, then -1.  accept_len excludes the root. */
int oracle_accept_n(const int32_t* draft_tok, const int32_t* parent, const int32_t* argmax,
                    const unsigned char* tag /* [S][B], 1 = spine child; or NULL */, const int32_t* n_nodes /* [S] or NULL */,
                    int S, int B, int32_t* path, int32_t* accept_len, int32_t* bonus) {
    for (int s = 0; s < S; ++s) {
        const int32_t* par = parent + (size_t)s * B;
        const int32_t* tok = draft_tok + (size_t)s * B;
        const int32_t* am = argmax + (size_t)s * B;
        int32_t* p = path + (size_t)s * B;
        const int n = nodes_of(n_nodes, s, B);             /* the walk sees the first n nodes only */
        if (n < 0) return -4;
        for (int j = 0; j < B; ++j) p[j] = -1;
        if (n == 0) {                                      /* the sequence has left the batch */
            accept_len[s] = 0;
            bonus[s] = -1;
            continue;
        }
        if (oracle_check_parent(par, n) != 0) return -1;
        int v = 0, len = 0;
        p[0] = 0;
        for (;;) {
            int next = -1;
            if (tag) {
                for (int c = v + 1; c < n && next < 0; ++c)      /* priority 1: spine child */
                    if (par[c] == v && tag[(size_t)s * B + c] && tok[c] == am[v]) next = c;
                for (int c = v + 1; c < n && next < 0; ++c)      /* priority 2: branch children */
                    if (par[c] == v && !tag[(size_t)s * B + c] && tok[c] == am[v]) next = c;
            } else {
                for (int c = v + 1; c < n && next < 0; ++c)
                    if (par[c] == v && tok[c] == am[v]) next = c;
            }
            if (next < 0) break;
            ++len;
            p[len] = next;
            v = next;
        }
        accept_len[s] = len;
        bonus[s] = am[v];
    }
    return 0;
}

int oracle_accept(const int32_t* draft_tok, const int32_t* parent, const int32_t* argmax,
                  const unsigned char* tag, int S, int B, int32_t* path, int32_t* accept_len, int32_t* bonus) {
    return oracle_accept_n(draft_tok, parent, argmax, tag, NULL, S, B, path, accept_len, bonus);
}

/* ------------------------------------------------------------------ KV compaction (out of place)
 * k_out/v_out start as copies of the caches; row ctx+j <- row ctx+path[j] of the ORIGINAL cache,
 * j = 0..accept_len.  new_ctx = ctx + 1 + accept_len.  Rows >= new_ctx are left as they were. */
int oracle_kv_compact_n(const uint16_t* kc, const uint16_t* vc, const int64_t* row_off, const int32_t* ctx_len,
                        const int32_t* path, const int32_t* accept_len, const int32_t* n_nodes /* [S] or NULL */,
                        int S, int B, int H, int D, uint16_t* k_out, uint16_t* v_out, int32_t* new_ctx) {
    size_t row_elems = (size_t)H * D;
    for (int s = 0; s < S; ++s) {
        const int n = nodes_of(n_nodes, s, B);
        if (n < 0) return -4;
        if (n == 0) { new_ctx[s] = ctx_len[s]; continue; }     /* left the batch: nothing moves, nothing is appended */
        int L = accept_len[s];
        if (L < 0 || L >= n) return -1;
        for (int j = 0; j <= L; ++j) {
            int src = path[(size_t)s * B + j];
            if (src < 0 || src >= n) return -1;
            size_t dst_row = (size_t)(row_off[s] + ctx_len[s] + j);
            size_t src_row = (size_t)(row_off[s] + ctx_len[s] + src);
            memcpy(k_out + dst_row * row_elems, kc + src_row * row_elems, row_elems * sizeof(uint16_t));
            memcpy(v_out + dst_row * row_elems, vc + src_row * row_elems, row_elems * sizeof(uint16_t));
        }
        new_ctx[s] = ctx_len[s] + 1 + L;
    }
    return 0;
}

int oracle_kv_compact(const uint16_t* kc, const uint16_t* vc, const int64_t* row_off, const int32_t* ctx_len,
                      const int32_t* path, const int32_t* accept_len, int S, int B, int H, int D,
                      uint16_t* k_out, uint16_t* v_out, int32_t* new_ctx) {
    return oracle_kv_compact_n(kc, vc, row_off, ctx_len, path, accept_len, NULL, S, B, H, D, k_out, v_out, new_ctx);
}

/* ------------------------------------------------------------------ logit harvest into the Tier-1 adjacency table
 * App. "Aggressive logit harvesting" + "Dense GPU bigram adjacency table" (Tier 1, unigram): two dense
 * [table_rows][k] tensors hold, for every vocabulary token, the ids and the "logit-derived scores" of its
 * top-k successors; every row of every forward's logits is harvested, rejected branches included.
 * Reading used here: row r of the logits predicts the successor of token row_tok[r]; its score is the softmax
 * probability exp(logit - lse_r), lse_r = log sum_j exp(logit_j) over the first V entries.  Rows are harvested in
 * order r = 0 .. rows-1, so when several rows carry the same token the LAST one is what the table keeps.
 * Rows whose token is outside [0, table_rows) are skipped.  row_lse [rows] may be NULL. */
int oracle_harvest(const uint16_t* logits, int rows, int V, int64_t ldl, int k, const int32_t* row_tok,
                   int table_rows, int32_t* adj_ids, double* adj_scores, double* row_lse) {
    if (k < 1 || k > V) return -1;
    vi_t* a = (vi_t*)malloc(sizeof(vi_t) * (size_t)V);
    if (!a) return -2;
    for (int r = 0; r < rows; ++r) {
        double mx = -INFINITY;
        for (int j = 0; j < V; ++j) {
            a[j].v = bf16_to_f64(logits[(size_t)r * ldl + j]);
            a[j].idx = j;
            if (a[j].v > mx) mx = a[j].v;
        }
        double sum = 0.0;
        for (int j = 0; j < V; ++j) sum += exp(a[j].v - mx);
        const double lse = mx + log(sum);
        if (row_lse) row_lse[r] = lse;
        const int tok = row_tok[r];
        if (tok < 0 || tok >= table_rows) continue;
        qsort(a, (size_t)V, sizeof(vi_t), cmp_vi);
        for (int j = 0; j < k; ++j) {
            adj_ids[(size_t)tok * k + j] = a[j].idx;
            adj_scores[(size_t)tok * k + j] = exp(a[j].v - lse);
        }
    }
    free(a);
    return 0;
}
