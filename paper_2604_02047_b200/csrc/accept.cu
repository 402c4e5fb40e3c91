// Greedy acceptance walk (Algorithm 3, UnifiedGreedyWalk): one warp per sequence.
//
// match[c] = (draft_tok[c] == argmax[parent[c]]) is evaluated for all nodes at once; the walk then
// repeatedly takes the lowest-index matching child of the current node (a warp min-reduction), which
// is the pointer walk of Algorithm 3 with "spine child before branch children" realised by the
// spine-first node order.  parent[] is validated first; an invalid tree yields neutral outputs and
// a status bit instead of a walk.
#include "goose_internal.cuh"

namespace goose {

__global__ void __launch_bounds__(32)
accept_kernel(const int32_t* __restrict__ draft_tok, const int32_t* __restrict__ parent,
              const int32_t* __restrict__ n_nodes, const int32_t* __restrict__ argmax, int B, int32_t* __restrict__ path,
              int32_t* __restrict__ accept_len, int32_t* __restrict__ bonus, int32_t* __restrict__ status) {
    const int s = blockIdx.x, lane = threadIdx.x;
    const int32_t* par = parent + (size_t)s * B;
    const int32_t* tok = draft_tok + (size_t)s * B;
    const int32_t* am = argmax + (size_t)s * B;
    int32_t* p = path + (size_t)s * B;
    pdl_wait();
    pdl_trigger();
    // the walk sees the first nn nodes of the tree; nn = 0: the sequence has left the batch (nothing of it is read)
    const int nn = nodes_of(n_nodes, s, B);
    if (nn == 0) {
        for (int c = lane; c < B; c += 32) p[c] = -1;
        if (lane == 0) {
            accept_len[s] = 0;
            bonus[s] = -1;
            if (nodes_bad(n_nodes, s, B)) atomicOr(&status[s], GOOSE_ST_BAD_NODES);
        }
        return;
    }

    constexpr int kPer = kMaxB / 32;
    int my_par[kPer];
    bool my_match[kPer];
    bool bad = false;
#pragma unroll
    for (int t = 0; t < kPer; ++t) {
        int c = lane + 32 * t;
        my_par[t] = -2;
        my_match[t] = false;
        if (c < nn) {
            int pp = par[c];
            my_par[t] = pp;
            if (c == 0) bad |= (pp != -1);
            else bad |= (pp < 0 || pp >= c);
        }
    }
    bad = __any_sync(0xFFFFFFFFu, bad);
    for (int c = lane; c < B; c += 32) p[c] = (c == 0) ? 0 : -1;
    if (bad) {
        if (lane == 0) {
            accept_len[s] = 0;
            bonus[s] = -1;
            atomicOr(&status[s], GOOSE_ST_BAD_PARENT);
        }
        return;
    }
#pragma unroll
    for (int t = 0; t < kPer; ++t) {
        int c = lane + 32 * t;
        if (c >= 1 && c < nn) my_match[t] = (tok[c] == am[my_par[t]]);
    }
    __syncwarp();
    int v = 0, len = 0;
    for (int step = 0; step < nn - 1; ++step) {
        int cand = 0x7FFFFFFF;
#pragma unroll
        for (int t = kPer - 1; t >= 0; --t)
            if (my_match[t] && my_par[t] == v) cand = lane + 32 * t;
        cand = __reduce_min_sync(0xFFFFFFFFu, cand);
        if (cand == 0x7FFFFFFF) break;
        ++len;
        if (lane == 0) p[len] = cand;
        v = cand;
    }
    if (lane == 0) {
        accept_len[s] = len;
        bonus[s] = am[v];
    }
}

cudaError_t launch_accept(goose_ctx* c, const int32_t* draft_tok, const int32_t* parent, const int32_t* n_nodes,
                          const int32_t* argmax, int S, int B, int32_t* path, int32_t* accept_len, int32_t* bonus,
                          cudaStream_t st) {
    if (S == 0) return cudaSuccess;
    cudaError_t e = launch_pdl(accept_kernel, dim3(S), dim3(32), 0, st, draft_tok, parent, n_nodes, argmax, B, path,
                               accept_len, bonus, c->status);
    c->launches++;
    return e;
}

}  // namespace goose
