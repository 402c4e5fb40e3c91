/*
 * goose.h -- C ABI of the B200 (sm_100a) tree-verification step of Goose.
 *
 * One verification step scores a spine tree of B draft tokens in a single pass
 * (Sec. 4, Stages 2-3; Algorithm 3):
 *   goose_tree_attn   tree-masked attention of the B draft queries over the prefix KV cache
 *                     plus each node's in-tree ancestors,
 *   goose_node_topk   per-node greedy argmax and top-k of the vocabulary logits,
 *   goose_accept      the greedy longest-accepted-path walk,
 *   goose_kv_compact  in-place compaction of the accepted nodes' K/V rows.
 *
 * Conventions (all entry points)
 *   - Every data pointer is a DEVICE pointer owned by the caller unless the argument is
 *     documented as "host".  The library owns only the workspace inside goose_ctx.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default
 *     stream), never synchronise the host, and return as soon as the work is enqueued.
 *     goose_verify_step_host and goose_last_status are the exceptions: they synchronise.
 *   - bf16 tensors are passed as void*; "bf16 [a][b]" means row-major, last index fastest.
 *   - Return value: GOOSE_OK, or a negative code.  Argument errors are detected on the host
 *     before anything is enqueued.  Data-dependent errors (an invalid parent[] array) are
 *     detected on the device: the affected sequence gets zero-filled / neutral outputs and a
 *     non-zero status word (goose_last_status); a kernel never traps and never spins without
 *     a bound.
 *   - A goose_ctx must not be used from two streams at once (its workspace is shared), and every call that takes
 *     a context must be made with the context's device current (cudaSetDevice), otherwise GOOSE_EINVAL;
 *     goose_verify_step_host, goose_last_status and goose_selftest_bounded_wait select the device themselves.
 *
 * Tree layout (Algorithm 1): node 0 is the anchor/root and counts towards B;
 * parent[0] = -1 and 0 <= parent[i] < i (topological order).  B <= GOOSE_MAX_B.
 *
 * KV cache layout: bf16 [kv_rows][H][D], token-major.  Sequence s owns rows
 * row_off[s] .. row_off[s] + ctx_len[s] + B - 1: first its ctx_len[s] prefix tokens, then the
 * K/V of tree node i at row row_off[s] + ctx_len[s] + i (written by the caller before the call).
 *
 * Per-sequence node counts.  The paper's batched prototype keeps finished requests in the batch as
 * padding and pays for them (App. "Batch-Size Sweep"); its Discussion leaves a production batched path
 * open.  Every call that takes a tree takes an optional device array n_nodes int32 [S] (NULL = every tree
 * has B nodes): sequence s has the nodes 0 .. n_nodes[s]-1 of its arrays (B stays the stride of q, out,
 * parent, draft_tok and of the logits rows).  Nodes i >= n_nodes[s] do not exist: their parent, token,
 * query, logits row and K/V row are never read (they may hold anything, NaN included), nothing is written
 * for them (out, lse, argmax, topk rows keep their contents; path entries are -1), and the sequence needs
 * only ctx_len[s] + n_nodes[s] cache rows.  The results for the nodes that exist are those of the tree
 * cut to its first n_nodes[s] nodes.  n_nodes[s] = 0 is a sequence that has left the batch: nothing of
 * it is read (row_off / ctx_len excepted) or moved; accept_len 0, bonus -1, path all -1,
 * new_ctx_len = ctx_len.  A value outside [0, B] is treated as 0 and sets GOOSE_ST_BAD_NODES.
 * The top-k then reads only the logits rows of nodes that exist (V * 2 bytes saved per absent node).
 * Trees padded by goose_pad_tree instead (n_nodes = NULL) are verified as B-node trees: the padding nodes'
 * K/V rows and logits rows ARE read then and must hold finite values.
 */
#ifndef GOOSE_H_
#define GOOSE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GOOSE_OK        0
#define GOOSE_EINVAL   (-1)   /* bad argument (null / misaligned pointer, size out of range)        */
#define GOOSE_ENOMEM   (-2)   /* workspace allocation failed                                       */
#define GOOSE_ECUDA    (-3)   /* a CUDA runtime / driver call failed; see goose_strerror           */
#define GOOSE_ETIMEOUT (-4)   /* a bounded device-side wait gave up (reported by goose_last_status) */

#define GOOSE_MAX_B     128   /* tree nodes per sequence (one 128-bit ancestor mask per node)      */
#define GOOSE_MAX_K      16   /* top-k width                                                       */
#define GOOSE_MAX_GROUP  16   /* query heads per key/value head (grouped-query attention)           */
#define GOOSE_HEAD_DIM  128   /* the only supported head dimension                                 */
#define GOOSE_MAX_V  262144   /* vocabulary size limit of goose_node_topk                          */
#define GOOSE_STATIC_TOPK_MAX_ROWS 2048   /* row limit of goose_node_topk_static                    */

/* per-sequence status bits (goose_last_status) */
#define GOOSE_ST_BAD_PARENT   1   /* parent[] is not a rooted tree in topological order */
#define GOOSE_ST_BAD_PATH     2   /* path[] / accept_len[] handed to goose_kv_compact is invalid */
#define GOOSE_ST_TIMEOUT      4   /* a device-side wait ran out of polls */
#define GOOSE_ST_BAD_ROWS     8   /* row_off[] / ctx_len[] put a sequence's rows outside [0, kv_rows): nothing moved */
#define GOOSE_ST_BAD_NODES   16   /* n_nodes[s] outside [0, B]: the sequence is treated as having left the batch */

/* attention kernel selection (goose_set_attn_impl) */
#define GOOSE_ATTN_AUTO  0
#define GOOSE_ATTN_MMA   1    /* warp-level mma.sync flash-decode kernel (any B <= 128)            */
#define GOOSE_ATTN_UMMA  2    /* tcgen05 + TMEM + TMA persistent kernel                            */

typedef struct goose_ctx goose_ctx;

/* Create a context on CUDA device `device`.  Allocates the workspace (split-KV partials,
 * arrival counters, per-sequence status) for up to max_S sequences of up to max_B <= 128 nodes
 * and max_H heads; head_dim must be 128.  *out is NULL on failure.                              */
int goose_create(goose_ctx** out, int device, int max_S, int max_B, int max_H, int head_dim);

/* Free the workspace.  The caller must have synchronised every stream that used the context.   */
int goose_destroy(goose_ctx* ctx);

/* Static description of a return code; for GOOSE_ECUDA the text of the last CUDA error seen
 * by this thread is appended.  The pointer stays valid until the next call from this thread.   */
const char* goose_strerror(int rc);

/* Choose the attention kernel (GOOSE_ATTN_*).  AUTO picks per call from B and the problem size. */
int goose_set_attn_impl(goose_ctx* ctx, int impl);

/* Tree attention (Sec. 4 Stage 1 "tree attention mask"; Algorithm 3 step 1).
 * For sequence s, head h, node i:  out[s][i][h][:] = softmax_j(scale * q[s][i][h] . K[j][h]) V[j][h]
 * over the visible keys j = prefix rows 0..ctx_len[s]-1 and tree rows ctx_len[s]+a for every
 * ancestor a of i, i included.  bf16 inputs, fp32 accumulation, bf16 output (round to nearest even).
 *   q        bf16 [S][B][H][D]                       16-byte aligned
 *   k_cache, v_cache  bf16 [kv_rows][H][D]           16-byte aligned; kv_rows = rows allocated
 *   row_off  int64 [S], ctx_len int32 [S], parent int32 [S][B], n_nodes int32 [S] or NULL   (device arrays)
 *   out      bf16 [S][B][H][D]; lse fp32 [S][B][H] = log-sum-exp of the scaled scores, or NULL
 * Rows row_off[s]+ctx_len[s]+B .. are never read as values (their contents may be anything).
 * ctx_len[s] = 0 is legal.  S <= max_S, B <= max_B, H <= max_H, D == 128, 0 < scale < 1e30.       */
int goose_tree_attn(goose_ctx* ctx, const void* q, const void* k_cache, const void* v_cache, int64_t kv_rows,
                    const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent, const int32_t* n_nodes,
                    int S, int B, int H, int D, float scale, void* out, float* lse, void* stream);

/* Same for grouped-query attention, the head layout of the 8B models of the paper's evaluation (Sec. 5 set-up: 32
 * query heads over 8 key/value heads): q and out have H heads, the caches Hkv heads, H a multiple of Hkv with
 * H / Hkv <= GOOSE_MAX_GROUP, and query head h reads key/value head h / (H / Hkv).
 *   k_cache, v_cache  bf16 [kv_rows][Hkv][D]
 * Hkv == H is goose_tree_attn.  The tensor-core kernel puts the H / Hkv query heads of a group into one tile, so the
 * key/value rows of a head are read once per group while B * (H / Hkv) <= 128, and once per
 * ceil(B / floor(128 / (H / Hkv))) otherwise.  Other arguments, limits and errors as goose_tree_attn.          */
int goose_tree_attn_gqa(goose_ctx* ctx, const void* q, const void* k_cache, const void* v_cache, int64_t kv_rows,
                        const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent, const int32_t* n_nodes,
                        int S, int B, int H, int Hkv, int D, float scale, void* out, float* lse, void* stream);

/* Per-node argmax and top-k (Algorithm 3 step 2; App. C.1 "aggressive logit harvesting": every
 * row of the forward's logits is harvested, rejected branches included).
 * For each of `rows` rows: the ids of the k largest of the first V values, ordered by
 * (value descending, index ascending); -0.0 equals +0.0; argmax[r] = topk_ids[r][0].
 *   logits bf16 [rows][ldl]  16-byte aligned, ldl % 8 == 0, ldl >= V, finite values
 *   1 <= k <= min(V, GOOSE_MAX_K); V <= GOOSE_MAX_V
 *   argmax int32 [rows]; topk_ids int32 [rows][k]; topk_vals fp32 [rows][k] (exact values) or NULL
 *   n_nodes int32 [rows / B] or NULL, with B (ignored when n_nodes is NULL; else rows % B == 0): row s * B + i
 *   is the row of node i of sequence s and is skipped -- not read, outputs untouched -- when i >= n_nodes[s]  */
int goose_node_topk(goose_ctx* ctx, const void* logits, int rows, int V, int64_t ldl, int k,
                    const int32_t* n_nodes, int B, int32_t* argmax, int32_t* topk_ids, float* topk_vals, void* stream);

/* Harvest of a forward's logits into the Tier-1 (unigram) adjacency table (App. C.1 "Aggressive logit
 * harvesting"; "Dense GPU bigram adjacency table", Tier 1: two dense |V| x K tensors with the ids and the
 * "logit-derived scores" of each token's top-K successors; every row is harvested, rejected branches and
 * prefill rows included).  Runs goose_node_topk with the row log-sum-exp, then for every row r writes
 *   adj_ids[row_tok[r]][j] = topk_ids[r][j],  adj_scores[row_tok[r]][j] = exp(topk_vals[r][j] - row_lse[r])
 * i.e. the softmax probability of the successor.  Rows are harvested in row order: of several rows with
 * the same token the last one is kept.  Rows whose token is outside [0, table_rows) are skipped; table
 * rows of tokens that do not occur keep their contents.
 *   row_tok int32 [rows]: the token whose successors row r predicts (a tree node's own draft token)
 *   adj_ids int32 [table_rows][k], adj_scores fp32 [table_rows][k]   (updated in place)
 *   argmax [rows], topk_ids [rows][k], topk_vals [rows][k], row_lse fp32 [rows]: outputs, all required       */
int goose_harvest(goose_ctx* ctx, const void* logits, int rows, int V, int64_t ldl, int k, const int32_t* row_tok,
                  int table_rows, int32_t* adj_ids, float* adj_scores, int32_t* argmax, int32_t* topk_ids,
                  float* topk_vals, float* row_lse, void* stream);

/* goose_node_topk without a context and without any allocation.  (The paper has no counterpart: this
 * entry point exists for integration reasons only.)
 * Some hosts may not allocate device memory once they are running: an inference server that plans all
 * of its device memory up front and treats a later cudaMalloc as an error, or a plug-in that is called
 * at a point where entering the allocator (and the implicit device synchronisation it can cause) is not
 * allowed.  goose_create allocates, so such callers cannot use goose_node_topk.  This variant computes
 * exactly the same result with the same kernel; its only scratch (the partial winners and arrival
 * counters used when the 32768-element chunks of a long row are handled by several thread blocks) is a
 * fixed array of about 2 MiB that is part of the library image, so every GPU that loads the library holds
 * it until the process exits.
 *   - Arguments, layouts and results as goose_node_topk, all data pointers on the CURRENT device;
 *     rows <= GOOSE_STATIC_TOPK_MAX_ROWS, otherwise GOOSE_EINVAL (nothing is enqueued).
 *   - It calls no cudaMalloc / cudaFree and no allocating library routine.  The first call on each
 *     device looks up the device address of the array (cudaGetSymbolAddress, with that device current),
 *     reads the device's multiprocessor count and sets the kernel's shared-memory attribute (host-side
 *     queries, made once per device).
 *   - All calls share the one array, which keeps the contents of the previous call; the counters it
 *     needs at zero are cleared on `stream` before the kernel.  Two calls whose kernels may overlap on
 *     the GPU (different streams, no dependency between them) race on the array: serialise them.
 *   - There is no status word behind this entry point: should one of the kernel's bounded waits run out (a
 *     copy that never completes), the call has already returned GOOSE_OK, the time-out is not reported, and
 *     the rows concerned keep whatever argmax / topk_ids / topk_vals held before.  Callers that need the
 *     report use goose_node_topk.                                                                        */
int goose_node_topk_static(const void* logits, int rows, int V, int64_t ldl, int k,
                           int32_t* argmax, int32_t* topk_ids, float* topk_vals, void* stream);

/* Greedy acceptance walk (Algorithm 3, UnifiedGreedyWalk).  From node 0, repeatedly move to the
 * child c of the current node v with draft_tok[c] == argmax[v]; stop when no child matches.
 * If sibling tokens are not distinct the matching child with the lowest index is taken.
 *   draft_tok, parent, argmax  int32 [S][B]; n_nodes int32 [S] or NULL
 *   path int32 [S][B]: path[s][0] = 0, then the accepted nodes in order, then -1
 *   accept_len int32 [S]: accepted draft nodes, root excluded; bonus int32 [S] = argmax at the last
 *   accepted node.  An invalid parent[] gives accept_len 0, path {0,-1,..}, bonus -1 and status.  */
int goose_accept(goose_ctx* ctx, const int32_t* draft_tok, const int32_t* parent, const int32_t* n_nodes,
                 const int32_t* argmax, int S, int B, int32_t* path, int32_t* accept_len, int32_t* bonus, void* stream);

/* KV compaction.  The paper does not describe cache handling after acceptance; this call keeps
 * the accepted nodes' rows in path order directly after the prefix, in place:
 * row ctx_len[s]+j <- row ctx_len[s]+path[s][j] for j = 0..accept_len[s], for K and V;
 * new_ctx_len[s] = ctx_len[s] + 1 + accept_len[s].  Rows >= new_ctx_len[s] are unspecified after
 * the call.  path must be increasing (as goose_accept produces it).  n_nodes int32 [S] or NULL: a
 * sequence with n_nodes[s] = 0 has left the batch (nothing moves, new_ctx_len[s] = ctx_len[s]).
 * new_ctx_len must not overlap ctx_len (GOOSE_EINVAL): every thread block of the launch reads ctx_len[s]
 * while one of them writes new_ctx_len[s].  To chain steps without a host round trip, alternate two
 * arrays: step t+1 takes step t's new_ctx_len as its ctx_len and writes the other array.             */
int goose_kv_compact(goose_ctx* ctx, void* k_cache, void* v_cache, int64_t kv_rows,
                     const int64_t* row_off, const int32_t* ctx_len, const int32_t* path,
                     const int32_t* accept_len, const int32_t* n_nodes, int S, int B, int H, int D,
                     int32_t* new_ctx_len, void* stream);

/* The whole step on one stream, in data-flow order: tree attention, node top-k (rows = S*B),
 * acceptance walk, KV compaction (the last two share one launch, which with the tensor-core attention
 * kernel also finishes the attention: the merge of its split heads runs there, beside the walk).  All
 * results, out and lse included, are complete in stream order when the call's last kernel is.  Arguments
 * and results as in the four calls above (new_ctx_len must not overlap ctx_len).  q, the caches' tree rows, parent, draft_tok,
 * logits, ctx_len and row_off are INPUTS of the step: they must be complete in stream order before the
 * call and nothing else may write them until the step is done; some kernels of the step read them
 * ahead of their stream-order dependency on the step's earlier kernels.                              */
int goose_verify_step(goose_ctx* ctx, const void* q, void* k_cache, void* v_cache, int64_t kv_rows,
                      const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent,
                      const int32_t* n_nodes, const int32_t* draft_tok, const void* logits, int64_t ldl,
                      int S, int B, int H, int D, int V, int k, float scale,
                      void* out, float* lse, int32_t* argmax, int32_t* topk_ids, float* topk_vals,
                      int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* new_ctx_len,
                      void* stream);

/* The whole step for grouped-query attention: attention as goose_tree_attn_gqa (q, out with H heads), compaction
 * over the caches' Hkv heads; everything else as goose_verify_step (which is this call with Hkv == H).       */
int goose_verify_step_gqa(goose_ctx* ctx, const void* q, void* k_cache, void* v_cache, int64_t kv_rows,
                          const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent,
                          const int32_t* n_nodes, const int32_t* draft_tok, const void* logits, int64_t ldl,
                          int S, int B, int H, int Hkv, int D, int V, int k, float scale,
                          void* out, float* lse, int32_t* argmax, int32_t* topk_ids, float* topk_vals,
                          int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* new_ctx_len,
                          void* stream);

/* The whole step plus the harvest of its logits (Algorithm 2: every cycle verifies a tree and harvests the forward's
 * logits, rejected branches included): as goose_verify_step_gqa, and additionally row_lse fp32 [S*B] and the update
 * of the adjacency table as in goose_harvest with row_tok = draft_tok (a node's logits row predicts the successor of
 * that node's own draft token; rows with a negative token, e.g. padding nodes, are skipped).  The logits are read
 * once: the top-k pass that feeds the acceptance walk also returns the log-sum-exp.  topk_vals is required.
 * With row_lse, adj_ids and adj_scores all NULL (table_rows ignored) this is goose_verify_step_gqa.             */
int goose_verify_step_harvest(goose_ctx* ctx, const void* q, void* k_cache, void* v_cache, int64_t kv_rows,
                              const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent,
                              const int32_t* n_nodes, const int32_t* draft_tok, const void* logits, int64_t ldl,
                              int S, int B, int H, int Hkv, int D, int V, int k, float scale,
                              void* out, float* lse, int32_t* argmax, int32_t* topk_ids, float* topk_vals,
                              int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* new_ctx_len,
                              float* row_lse, int table_rows, int32_t* adj_ids, float* adj_scores, void* stream);

/* Host-buffer variant of the whole step (the end-to-end call).  The prefix KV cache stays on the
 * device (k_cache / v_cache are device pointers, state carried from step to step); everything a
 * step consumes or produces is in HOST memory (pinned memory makes the copies asynchronous):
 *   in : h_q bf16 [S][B][H][D]; h_k_new, h_v_new bf16 [S][B][H][D] = the tree nodes' K/V rows,
 *        copied to rows row_off[s]+ctx_len[s]+i; h_row_off int64 [S]; h_ctx_len int32 [S];
 *        h_parent, h_draft_tok int32 [S][B]; h_n_nodes int32 [S] or NULL (validated on the host: outside
 *        [0, B] is GOOSE_EINVAL; only the K/V rows of nodes that exist are copied; the output arrays are
 *        copied back whole, so the output rows of nodes that do not exist are unspecified here);
 *        h_logits bf16 [S*B][V] (dense, ldl = V)
 *   out: h_out bf16 [S][B][H][D]; h_argmax [S*B]; h_topk_ids [S*B][k]; h_topk_vals [S*B][k] or NULL;
 *        h_path [S][B]; h_accept_len, h_bonus, h_new_ctx_len [S]
 * Copies in, runs goose_verify_step, copies out, and synchronises `stream` before returning.
 * The logits (most of the bytes, needed by the top-k only) are uploaded on a stream of the context's own while the
 * attention kernels run, and h_out is copied down on another one as soon as the attention is done; the small arrays
 * travel through one pinned block of the context, one copy each way.
 * Device and pinned staging buffers, those streams and their events are created inside the context on first use and
 * grow on demand; calls on one context must not overlap.                                                     */
int goose_verify_step_host(goose_ctx* ctx, void* k_cache, void* v_cache, int64_t kv_rows,
                           const void* h_q, const void* h_k_new, const void* h_v_new,
                           const int64_t* h_row_off, const int32_t* h_ctx_len,
                           const int32_t* h_parent, const int32_t* h_n_nodes, const int32_t* h_draft_tok, const void* h_logits,
                           int S, int B, int H, int D, int V, int k, float scale,
                           void* h_out, int32_t* h_argmax, int32_t* h_topk_ids, float* h_topk_vals,
                           int32_t* h_path, int32_t* h_accept_len, int32_t* h_bonus,
                           int32_t* h_new_ctx_len, void* stream);

/* Host-buffer variant of goose_verify_step_gqa: as goose_verify_step_host, with h_q / h_out of H heads and
 * h_k_new, h_v_new bf16 [S][B][Hkv][D] (rows of the Hkv-head caches).                                        */
int goose_verify_step_host_gqa(goose_ctx* ctx, void* k_cache, void* v_cache, int64_t kv_rows,
                               const void* h_q, const void* h_k_new, const void* h_v_new,
                               const int64_t* h_row_off, const int32_t* h_ctx_len,
                               const int32_t* h_parent, const int32_t* h_n_nodes, const int32_t* h_draft_tok,
                               const void* h_logits, int S, int B, int H, int Hkv, int D, int V, int k, float scale,
                               void* h_out, int32_t* h_argmax, int32_t* h_topk_ids, float* h_topk_vals,
                               int32_t* h_path, int32_t* h_accept_len, int32_t* h_bonus,
                               int32_t* h_new_ctx_len, void* stream);

/* ---- host routines of the loop around the verification step (all pointers below are HOST pointers) ---- */

/* BuildSpineTree (Algorithm 1).  anchor = the last accepted token (spine root); chain[m] = the context-match
 * draft; adj_ids int32 [table_rows][K] = Tier-1 adjacency table ids in rank order (negative = empty slot).
 * Budget: b_s = min(m, floor(B r)), b_r = floor((B-1-b_s)(1-rho)), b_rho = B-1-b_s-b_r; step 1 lays the spine,
 * step 2 attaches up to b_r ranked successors of the anchor to the root, step 3 attaches
 * a_i = floor(b_rho (1/i) / H_{b_s}) successors of spine token d_i to spine node i, step 4 extends every branch leaf
 * breadth-first by its top successor up to D nodes per branch while nodes remain.  Successors that would
 * duplicate a sibling (e.g. the spine continuation) are skipped.  Output in spine-first topological order
 * (parent[i] < i): draft_tok, parent (capacity B), is_spine (may be NULL), *n_nodes <= B, *n_spine = b_s + 1.  */
int goose_build_spine_tree(int32_t anchor, const int32_t* chain, int m, const int32_t* adj_ids, int table_rows, int K,
                           int B, int D, float r, float rho, int32_t* draft_tok, int32_t* parent, uint8_t* is_spine,
                           int32_t* n_nodes, int32_t* n_spine);

/* Fill nodes n_nodes..B-1 with padding (children of the root with negative tokens, which no argmax can match), so
 * that a tree with fewer than B nodes can be verified as a B-node tree (n_nodes = NULL in the calls above).  The
 * padding nodes' K/V rows and logits rows are then read like any other node's and must hold finite values (a
 * padding key gets weight 0 in the softmax of every real node, and 0 x NaN is NaN).  Passing the node count in
 * n_nodes[] instead needs no padding, reads none of those rows and leaves no such requirement.                  */
int goose_pad_tree(int32_t* draft_tok, int32_t* parent, int n_nodes, int B);

/* ContextMatch (paragraph after Algorithm 2): n-gram lookup with n in {5, 4, 3} of the last n tokens of ctx at
 * their most recent earlier occurrence; chain = the continuation (at most max_len tokens) of the longest n that
 * matched, *chain_len = 0 if none; *consensus = 1 iff at least two n's matched and agree on the first
 * continuation token.                                                                                           */
int goose_context_match(const int32_t* ctx, int n_ctx, int max_len, int32_t* chain, int32_t* chain_len,
                        int32_t* consensus);

/* Spine-ratio tier (hyper-parameter table): p_hat < 0.2 -> 0.15, < 0.4 -> 0.30, otherwise 0.50.                  */
float goose_spine_ratio_tier(float p_hat);

/* EMA of the spine acceptance rate, coefficient 0.3: 0.7 p_hat + 0.3 accepted/drafted (unchanged if drafted = 0). */
float goose_spine_ema(float p_hat, int accepted_spine, int drafted_spine);

/* Synchronise the device, copy the per-sequence status words (GOOSE_ST_* bits, OR-ed over all
 * calls since the last query) into host_status[0..S) (a HOST array) and clear them.
 * Returns GOOSE_ETIMEOUT if any word has GOOSE_ST_TIMEOUT set.  For tests and debugging.
 * Recovery rule: a call whose kernel timed out leaves its outputs incomplete and the context's cross-block
 * arrival counters half counted; this query is what resets them, so after a GOOSE_ST_TIMEOUT call it once
 * before the context is used again.                                                               */
int goose_last_status(goose_ctx* ctx, int32_t* host_status, int S);

/* Self-test of the device-side time-out path.  Runs a one-warp kernel whose wait (the same bounded mbarrier wait
 * the attention kernel uses) can never be satisfied and gives up after `limit_cycles` SM cycles (keep it short, e.g.
 * 1e6 = about half a millisecond).  Returns GOOSE_OK when the wait reported failure and the kernel returned
 * normally; afterwards goose_last_status shows GOOSE_ST_TIMEOUT in word 0 (and returns GOOSE_ETIMEOUT), and the
 * context remains fully usable.  Synchronises `stream`.                                                         */
int goose_selftest_bounded_wait(goose_ctx* ctx, int64_t limit_cycles, void* stream);

/* Number of kernels this library has launched through `ctx` since it was created.              */
int64_t goose_launch_count(goose_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* GOOSE_H_ */
