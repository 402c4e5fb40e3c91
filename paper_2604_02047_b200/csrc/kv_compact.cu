// In-place KV compaction of the accepted path (the paper leaves cache handling after acceptance
// implicit; the accepted nodes' rows are kept, in path order, directly after the prefix).
//
// Row ctx+j <- row ctx+path[j].  path is increasing with path[j] >= j, so a thread that owns one
// 16-byte column of the row and walks j upwards never overwrites a row it still has to read:
// sources of later moves are > j.  Moves are issued in batches of 8 (all loads of a batch before its
// stores; a batch's destinations are below every later source), which keeps 8 loads in flight per
// thread without any barrier.
#include "goose_internal.cuh"
#include "tree_attn_combine.cuh"

namespace goose {

constexpr int kCompactThreads = 128;
constexpr int kCompactBatch = 8;

// kCounts = false is the instantiation for n_nodes == NULL
template <bool kCounts>
__global__ void __launch_bounds__(kCompactThreads)
kv_compact_kernel(__nv_bfloat16* kc, __nv_bfloat16* vc,
                  const int64_t* __restrict__ row_off, const int32_t* __restrict__ ctx_len,
                  const int32_t* __restrict__ path, const int32_t* __restrict__ accept_len,
                  const int32_t* __restrict__ n_nodes,
                  int B, int row_vec /* 16-byte vectors per row = H*128*2/16 */, int64_t kv_rows,
                  int32_t* __restrict__ new_ctx, int32_t* __restrict__ status) {
    if (!kCounts) n_nodes = nullptr;

    __shared__ int s_path[kMaxB];
    __shared__ int s_bad;
    const int s = blockIdx.z;
    const int which = blockIdx.y;                        // 0 = K, 1 = V
    const int col = blockIdx.x * kCompactThreads + threadIdx.x;
    pdl_wait();
    pdl_trigger();
    const int ctx = ctx_len[s];
    const int nn = nodes_of(n_nodes, s, B);              // nodes of this sequence's tree; 0: it has left the batch
    if (nn == 0) {                                       // nothing moves, nothing is appended
        if (blockIdx.x == 0 && which == 0 && threadIdx.x == 0) {
            new_ctx[s] = ctx;
            if (nodes_bad(n_nodes, s, B)) atomicOr(&status[s], GOOSE_ST_BAD_NODES);
        }
        return;
    }
    int L = accept_len[s];
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    // rows this sequence owns must lie inside the cache: never form an address from unchecked device data
    const int64_t r0 = row_off[s];
    const bool bad_rows = ctx < 0 || r0 < 0 || r0 + ctx + nn > kv_rows;
    bool bad = (L < 0 || L >= nn) || bad_rows;
    if (!bad) {
        for (int j = threadIdx.x; j <= L; j += kCompactThreads) {
            int pj = path[(size_t)s * B + j];
            s_path[j] = pj;
            int prev = (j == 0) ? -1 : path[(size_t)s * B + j - 1];
            if (pj < j || pj >= nn || pj <= prev || (j == 0 && pj != 0)) s_bad = 1;
        }
    }
    __syncthreads();
    bad = bad || s_bad;
    if (bad) L = 0;
    if (blockIdx.x == 0 && which == 0 && threadIdx.x == 0) {
        new_ctx[s] = ctx + 1 + L;
        if (bad) atomicOr(&status[s], bad_rows ? GOOSE_ST_BAD_ROWS : GOOSE_ST_BAD_PATH);
    }
    if (bad || col >= row_vec) return;

    uint4* base = reinterpret_cast<uint4*>(which ? vc : kc) + ((size_t)(row_off[s] + ctx)) * row_vec + col;
    for (int j0 = 1; j0 <= L; j0 += kCompactBatch) {
        uint4 r[kCompactBatch];
#pragma unroll
        for (int t = 0; t < kCompactBatch; ++t) {
            int j = j0 + t;
            if (j <= L && s_path[j] != j) r[t] = base[(size_t)s_path[j] * row_vec];
        }
#pragma unroll
        for (int t = 0; t < kCompactBatch; ++t) {
            int j = j0 + t;
            if (j <= L && s_path[j] != j) base[(size_t)j * row_vec] = r[t];
        }
    }
}

cudaError_t launch_kv_compact(goose_ctx* c, __nv_bfloat16* kc, __nv_bfloat16* vc, const int64_t* row_off,
                              const int32_t* ctx_len, const int32_t* path, const int32_t* accept_len, const int32_t* n_nodes,
                              int S, int B, int H, int64_t kv_rows, int32_t* new_ctx, cudaStream_t st) {
    if (S == 0) return cudaSuccess;
    int row_vec = H * kHeadDim * 2 / 16;
    dim3 grid((row_vec + kCompactThreads - 1) / kCompactThreads, 2, S);
    cudaError_t e = launch_pdl(n_nodes ? kv_compact_kernel<true> : kv_compact_kernel<false>, grid, dim3(kCompactThreads), 0, st, kc, vc, row_off, ctx_len, path,
                               accept_len, n_nodes, B, row_vec, kv_rows, new_ctx, c->status);
    c->launches++;
    return e;
}

// ---------------------------------------------------------------------------------------------------
// Fused form used by goose_verify_step: the acceptance walk (Algorithm 3) and the compaction in one launch.
// Every CTA redoes the walk of its sequence with warp 0 (a handful of warp reductions) instead of waiting for
// a separate kernel; CTA (0, 0, s) publishes path / accept_len / bonus / new_ctx.
// parent[], draft_tok[], ctx_len[] and row_off[] are inputs of the step, complete before its first kernel started, so
// they are read before the dependency wait; argmax[] (the top-k kernel's result) and the cache rows are read after it.
// With a harvest (adj_ids != NULL) the launch carries a third block role, blockIdx.y == 2: one warp per logits row of the
// sequence writes that row's top-k ids and softmax scores to adjacency-table row draft_tok[row] unless a later row of the
// call carries the same token -- the rule of harvest_scatter_kernel, decided here before the wait (tokens are inputs).
// With the tensor-core attention kernel the launch also carries the merge of that kernel's split heads (kMerge: 0 = no
// merge role, 1 = multi-head, 2 = grouped-query attention; 256 threads per CTA then): blockIdx.y >= base_roles is head
// blockIdx.y - base_roles of the attention work list, blockIdx.x its group of 32 rows.  The merge needs the main kernel
// to be complete, which this launch's dependency wait implies (every CTA of the top-k kernel in between has waited for
// it), and nothing of the walk: it simply runs beside it instead of standing between the attention kernel and the top-k.
template <bool kCounts, int kMerge>
__global__ void __launch_bounds__(kMerge ? kCombineThreads : kCompactThreads)
accept_compact_kernel(__nv_bfloat16* kc, __nv_bfloat16* vc, const int64_t* __restrict__ row_off,
                      const int32_t* __restrict__ ctx_len, const int32_t* __restrict__ draft_tok,
                      const int32_t* __restrict__ parent, const int32_t* __restrict__ n_nodes,
                      const int32_t* __restrict__ argmax,
                      int B, int row_vec, int64_t kv_rows, int32_t* __restrict__ path,
                      int32_t* __restrict__ accept_len, int32_t* __restrict__ bonus, int32_t* __restrict__ new_ctx,
                      int32_t* __restrict__ status,
                      int rows_total, int table_rows, int k, const int32_t* __restrict__ topk_ids,
                      const float* __restrict__ topk_vals, const float* __restrict__ row_lse,
                      int32_t* __restrict__ adj_ids, float* __restrict__ adj_scores,
                      int base_roles, int merge_row_groups, const CombineArgs ca) {
    if (!kCounts) n_nodes = nullptr;
    constexpr int kT = kMerge ? kCombineThreads : kCompactThreads;   // threads of this launch
    if (kMerge && (int)blockIdx.y >= base_roles) {
        // ---- merge role: 32 rows of one head of the attention work list (the partials of the step's main kernel)
        if ((int)blockIdx.x >= merge_row_groups) {      // the grid is as wide as its widest role
            pdl_wait();
            pdl_trigger();
            return;
        }
        combine_heads<kMerge == 2, kCounts>(ca, blockIdx.x, (int)blockIdx.y - base_roles, blockIdx.z);
        return;
    }

    __shared__ int s_path[kMaxB];
    __shared__ int s_len;
    const int s = blockIdx.z;
    // n_nodes[] is an input of the step like parent[] and the tokens: read ahead of the wait.  nn = nodes of this
    // sequence's tree; 0: the sequence has left the batch and nothing of it is read or moved.
    const int nn = kCounts ? nodes_of(n_nodes, s, B) : B;
    const bool live = !kCounts || nn > 0;               // (without counts every sequence has its B nodes)
    if (blockIdx.y == 2) {
        // ---- harvest scatter role
        const int lane = threadIdx.x & 31;
        const int i = blockIdx.x * (kT / 32) + (threadIdx.x >> 5);   // node of sequence s
        const size_t r = (size_t)s * B + i;
        int tok = -1;
        bool write = false;
        if (i < nn) {
            tok = draft_tok[r];
            if (tok >= 0 && tok < table_rows) {
                bool later = false;                        // does a later row (of a node that exists) carry the same token?
                for (int j = (int)r + 1 + lane; j < rows_total; j += 32) {
                    if (!kCounts) { later |= (draft_tok[j] == tok); continue; }
                    const int sj = j / B;
                    if (j - sj * B < nodes_of(n_nodes, sj, B)) later |= (draft_tok[j] == tok);
                }
                write = !__any_sync(0xFFFFFFFFu, later);
            }
        }
        pdl_wait();
        pdl_trigger();
        if (write && lane < k) {
            adj_ids[(size_t)tok * k + lane] = topk_ids[r * k + lane];
            adj_scores[(size_t)tok * k + lane] = expf(topk_vals[r * k + lane] - row_lse[r]);
        }
        return;
    }
    if ((int)blockIdx.x * kT >= row_vec) {   // the grid is as wide as its widest role: nothing to copy here
        pdl_wait();
        pdl_trigger();
        return;
    }
    const int which = blockIdx.y;                        // 0 = K, 1 = V
    const int col = blockIdx.x * kT + threadIdx.x;
    const bool publisher = blockIdx.x == 0 && which == 0;
    // rows this sequence owns must lie inside the cache: never form an address from unchecked device data
    const int ctx0 = ctx_len[s];
    const int64_t r0 = row_off[s];
    const bool bad_rows = live && (ctx0 < 0 || r0 < 0 || r0 + ctx0 + nn > kv_rows);
    constexpr int kPer = kMaxB / 32;
    int my_par[kPer], my_tok[kPer];
    bool bad = false;
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        const int32_t* par = parent + (size_t)s * B;
        const int32_t* tok = draft_tok + (size_t)s * B;
#pragma unroll
        for (int t = 0; t < kPer; ++t) {
            const int c = lane + 32 * t;
            my_par[t] = -2;
            my_tok[t] = -1;
            if (c < nn) {
                const int pp = par[c];
                my_par[t] = pp;
                my_tok[t] = tok[c];
                bad |= (c == 0) ? (pp != -1) : (pp < 0 || pp >= c);
            }
        }
        bad = __any_sync(0xFFFFFFFFu, bad);
        for (int c = lane; c < B; c += 32) s_path[c] = (c == 0 && live) ? 0 : -1;
    }
    pdl_wait();
    pdl_trigger();
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        const int32_t* am = argmax + (size_t)s * B;
        bool my_match[kPer];
#pragma unroll
        for (int t = 0; t < kPer; ++t) my_match[t] = false;
        __syncwarp();
        int v = 0, len = 0;
        if (!bad && live) {
#pragma unroll
            for (int t = 0; t < kPer; ++t) {
                const int c = lane + 32 * t;
                if (c >= 1 && c < nn) my_match[t] = (my_tok[t] == am[my_par[t]]);
            }
            for (int step = 0; step < nn - 1; ++step) {
                int cand = 0x7FFFFFFF;
#pragma unroll
                for (int t = kPer - 1; t >= 0; --t)
                    if (my_match[t] && my_par[t] == v) cand = lane + 32 * t;
                cand = __reduce_min_sync(0xFFFFFFFFu, cand);
                if (cand == 0x7FFFFFFF) break;
                ++len;
                if (lane == 0) s_path[len] = cand;
                v = cand;
            }
        }
        __syncwarp();
        if (lane == 0) s_len = len;
        if (publisher) {
            for (int c = lane; c < B; c += 32) path[(size_t)s * B + c] = s_path[c];
            if (lane == 0) {
                accept_len[s] = len;
                bonus[s] = (bad || !live) ? -1 : am[v];
                new_ctx[s] = !live ? ctx0 : ctx0 + 1 + len;
                if (bad) atomicOr(&status[s], GOOSE_ST_BAD_PARENT);
                if (bad_rows) atomicOr(&status[s], GOOSE_ST_BAD_ROWS);
                if (kCounts && nodes_bad(n_nodes, s, B)) atomicOr(&status[s], GOOSE_ST_BAD_NODES);
            }
        }
    }
    __syncthreads();
    const int L = s_len;
    if (col >= row_vec || bad_rows) return;
    uint4* base = reinterpret_cast<uint4*>(which ? vc : kc) + ((size_t)(r0 + ctx0)) * row_vec + col;
    for (int j0 = 1; j0 <= L; j0 += kCompactBatch) {
        uint4 r[kCompactBatch];
#pragma unroll
        for (int t = 0; t < kCompactBatch; ++t) {
            const int j = j0 + t;
            if (j <= L && s_path[j] != j) r[t] = base[(size_t)s_path[j] * row_vec];
        }
#pragma unroll
        for (int t = 0; t < kCompactBatch; ++t) {
            const int j = j0 + t;
            if (j <= L && s_path[j] != j) base[(size_t)j * row_vec] = r[t];
        }
    }
}

cudaError_t launch_accept_compact(goose_ctx* c, __nv_bfloat16* kc, __nv_bfloat16* vc, const int64_t* row_off,
                                  const int32_t* ctx_len, const int32_t* draft_tok, const int32_t* parent,
                                  const int32_t* n_nodes, const int32_t* argmax, int S, int B, int H, int64_t kv_rows, int32_t* path,
                                  int32_t* accept_len, int32_t* bonus, int32_t* new_ctx, cudaStream_t st,
                                  int table_rows, int k, const int32_t* topk_ids, const float* topk_vals,
                                  const float* row_lse, int32_t* adj_ids, float* adj_scores, const CombinePlan* merge) {
    if (S == 0) return cudaSuccess;
    const bool with_merge = merge && merge->valid;     // the attention merge of this step rides in this launch
    const int threads = with_merge ? kCombineThreads : kCompactThreads;
    int row_vec = H * kHeadDim * 2 / 16;
    int gx = (row_vec + threads - 1) / threads;
    const bool scatter = adj_ids != nullptr;
    if (scatter) {
        const int sx = (B + threads / 32 - 1) / (threads / 32);   // one warp per logits row
        if (sx > gx) gx = sx;
    }
    const int base_roles = scatter ? 3 : 2;
    CombineArgs ca{};
    int merge_rg = 0, roles = base_roles;
    if (with_merge) {
        ca = merge->args; merge_rg = merge->row_groups; roles += ca.Hw;
        if (merge_rg > gx) gx = merge_rg;
    }
    dim3 grid(gx, roles, S);
    const bool counts = n_nodes != nullptr;
    const int mode = !with_merge ? 0 : (merge->grouped ? 2 : 1);
    auto kernel = mode == 0 ? (counts ? accept_compact_kernel<true, 0> : accept_compact_kernel<false, 0>)
                : mode == 1 ? (counts ? accept_compact_kernel<true, 1> : accept_compact_kernel<false, 1>)
                            : (counts ? accept_compact_kernel<true, 2> : accept_compact_kernel<false, 2>);
    cudaError_t e = launch_pdl(kernel, grid, dim3(threads), 0, st, kc, vc, row_off, ctx_len,
                               draft_tok, parent, n_nodes, argmax, B, row_vec, kv_rows, path, accept_len, bonus, new_ctx, c->status,
                               S * B, table_rows, k, topk_ids, topk_vals, row_lse, adj_ids, adj_scores,
                               base_roles, merge_rg, ca);
    c->launches++;
    return e;
}

}  // namespace goose
