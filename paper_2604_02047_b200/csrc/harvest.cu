// Harvest of a forward's logits into the Tier-1 (unigram) adjacency table (App. "Aggressive logit harvesting";
// "Dense GPU bigram adjacency table", Tier 1): for every logits row r the k best successor ids and their
// softmax probabilities exp(logit - lse_r) overwrite row row_tok[r] of the two dense [table_rows][k] tensors.
// Rows are harvested in row order, so of several rows that carry the same token the last one wins; the
// scatter kernel decides that per row by scanning the later rows' tokens (one warp per row, no atomics), which
// keeps the result independent of scheduling.  The top-k and the log-sum-exp come from node_topk_kernel.
#include "goose_internal.cuh"

namespace goose {

constexpr int kScatterThreads = 128;

__global__ void __launch_bounds__(kScatterThreads)
harvest_scatter_kernel(const int32_t* __restrict__ row_tok, int rows, int table_rows, int k,
                       const int32_t* __restrict__ ids, const float* __restrict__ vals,
                       const float* __restrict__ row_lse, int32_t* __restrict__ adj_ids,
                       float* __restrict__ adj_scores) {
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * (kScatterThreads / 32) + (threadIdx.x >> 5);
    pdl_wait();
    pdl_trigger();
    if (r >= rows) return;
    const int tok = row_tok[r];
    if (tok < 0 || tok >= table_rows) return;              // not a table row: skipped
    bool later = false;                                      // does a later row carry the same token?
    for (int j = r + 1 + lane; j < rows; j += 32) later |= (row_tok[j] == tok);
    if (__any_sync(0xFFFFFFFFu, later)) return;
    if (lane < k) {
        adj_ids[(size_t)tok * k + lane] = ids[(size_t)r * k + lane];
        adj_scores[(size_t)tok * k + lane] = expf(vals[(size_t)r * k + lane] - row_lse[r]);
    }
}

cudaError_t launch_harvest_scatter(goose_ctx* c, const int32_t* row_tok, int rows, int table_rows, int k,
                                   const int32_t* ids, const float* vals, const float* row_lse,
                                   int32_t* adj_ids, float* adj_scores, cudaStream_t st) {
    if (rows == 0) return cudaSuccess;
    dim3 grid((rows + kScatterThreads / 32 - 1) / (kScatterThreads / 32));
    cudaError_t e = launch_pdl(harvest_scatter_kernel, grid, dim3(kScatterThreads), 0, st, row_tok, rows, table_rows, k,
                               ids, vals, row_lse, adj_ids, adj_scores);
    c->launches++;
    return e;
}

}  // namespace goose
