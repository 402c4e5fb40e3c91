// Internal declarations shared by the CUDA translation units of libgoose.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "goose.h"

namespace goose {

constexpr int kHeadDim = GOOSE_HEAD_DIM;
constexpr int kMaxB = GOOSE_MAX_B;
constexpr int kMaxK = GOOSE_MAX_K;

// Workspace slot of one split-KV partial.  The mma kernel stores O fp32 [kMaxB][128] (unnormalised), then m[kMaxB],
// l[kMaxB]; the tcgen05 kernel uses the first half of a slot for its fp16 layout (see tree_attn_umma.cu).
constexpr int kPartialFloats = kMaxB * kHeadDim + 2 * kMaxB;

}  // namespace goose

struct goose_ctx {
    int device;
    int num_sms;
    int max_S, max_B, max_H;
    int attn_impl;            // GOOSE_ATTN_*
    // attention workspace
    float* partials;          // [n_slots][kPartialFloats]
    int n_slots;
    int32_t* head_counters;   // [max_S * max_H], zero between launches
    // top-k workspace
    unsigned long long* topk_cand;   // [topk_rows_cap][topk_chunks_cap][kMaxK]
    int32_t* row_counters;    // [topk_rows_cap]
    float* topk_lse_ws;       // [topk_rows_cap][chunks][2]: per-chunk (max, sum) of the log-sum-exp
    int64_t topk_cand_cap;    // elements
    int topk_rows_cap;
    // per-sequence status words
    int32_t* status;          // [max_S]
    int32_t* selftest_word;   // result word of goose_selftest_bounded_wait
    // host staging for goose_verify_step_host
    void* stage;              // device buffer
    size_t stage_bytes;
    void* pin;                // pinned host block: the small input arrays go up, the small results come down, in one copy each
    size_t pin_bytes;
    cudaStream_t side;        // the logits are uploaded here, next to the attention kernels
    cudaStream_t side_down;   // the attention output goes down here while the logits are still going up
    cudaEvent_t ev_fork, ev_logits, ev_attn, ev_out;
    long long launches;
    void* encode_tiled;       // cuTensorMapEncodeTiled entry point (driver), resolved at create
};

namespace goose {

// Programmatic dependent launch.  Every kernel of the library is launched with the
// programmatic-stream-serialisation attribute and runs  prologue (no global memory access) ->
// pdl_wait() -> pdl_trigger() -> body.  pdl_wait() returns once the preceding kernel in the stream has
// completed and its writes are visible; because that kernel passed its own pdl_wait() before it
// triggered, completion is transitive over the whole stream.  The overlap gained is the launch latency
// and the prologue of the next kernel.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Nodes of sequence s: n_nodes[s] when the array is given, else B.  The array is device data: a value outside [0, B]
// reads as 0 (the sequence is skipped like one that has left the batch) and is reported as GOOSE_ST_BAD_NODES.
__device__ __forceinline__ int nodes_of(const int32_t* __restrict__ n_nodes, int s, int B) {
    if (!n_nodes) return B;
    const int n = n_nodes[s];
    return (n < 0 || n > B) ? 0 : n;
}
__device__ __forceinline__ bool nodes_bad(const int32_t* __restrict__ n_nodes, int s, int B) {
    return n_nodes != nullptr && (n_nodes[s] < 0 || n_nodes[s] > B);
}

// Bounded mbarrier wait, shared by every kernel that waits on asynchronous copies or tensor-core commits.
// Returns 0 when the barrier phase completed, 1 when `*abort_flag` was raised by another thread of the CTA meanwhile,
// 2 when `limit_cycles` SM cycles passed (the caller raises the flag, records GOOSE_ST_TIMEOUT and unwinds).
__device__ __forceinline__ bool mbar_try_wait_parity(unsigned long long* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ int mbar_wait_bounded(unsigned long long* bar, uint32_t parity, long long limit_cycles,
                                                 volatile int* abort_flag) {
    if (mbar_try_wait_parity(bar, parity)) return 0;
    const long long t0 = clock64();
    for (;;) {
        if (*abort_flag) return 1;
        if (mbar_try_wait_parity(bar, parity)) return 0;
        if (clock64() - t0 > limit_cycles) return 2;
    }
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// launchers (each returns a cudaError_t from the launch)
// inputs_ready: the logits were complete before the kernel preceding this one in the stream started (see the kernel)
// n_nodes (may be NULL) with B: row r = s * B + i exists iff i < n_nodes[s]; other rows are neither read nor written
cudaError_t launch_node_topk(goose_ctx* c, const __nv_bfloat16* logits, int rows, int V, int64_t ldl, int k,
                             int32_t* argmax, int32_t* ids, float* vals, float* row_lse, cudaStream_t st,
                             bool inputs_ready = false, const int32_t* n_nodes = nullptr, int B = 0);
cudaError_t launch_harvest_scatter(goose_ctx* c, const int32_t* row_tok, int rows, int table_rows, int k,
                                   const int32_t* ids, const float* vals, const float* row_lse,
                                   int32_t* adj_ids, float* adj_scores, cudaStream_t st);
cudaError_t launch_accept(goose_ctx* c, const int32_t* draft_tok, const int32_t* parent, const int32_t* n_nodes,
                          const int32_t* argmax, int S, int B, int32_t* path, int32_t* accept_len, int32_t* bonus,
                          cudaStream_t st);
cudaError_t launch_kv_compact(goose_ctx* c, __nv_bfloat16* kc, __nv_bfloat16* vc, const int64_t* row_off,
                              const int32_t* ctx_len, const int32_t* path, const int32_t* accept_len, const int32_t* n_nodes,
                              int S, int B, int H, int64_t kv_rows, int32_t* new_ctx, cudaStream_t st);
cudaError_t launch_accept_compact(goose_ctx* c, __nv_bfloat16* kc, __nv_bfloat16* vc, const int64_t* row_off,
                                  const int32_t* ctx_len, const int32_t* draft_tok, const int32_t* parent,
                                  const int32_t* n_nodes, const int32_t* argmax, int S, int B, int H, int64_t kv_rows, int32_t* path,
                                  int32_t* accept_len, int32_t* bonus, int32_t* new_ctx, cudaStream_t st,
                                  int table_rows = 0, int k = 0, const int32_t* topk_ids = nullptr,
                                  const float* topk_vals = nullptr, const float* row_lse = nullptr,
                                  int32_t* adj_ids = nullptr, float* adj_scores = nullptr,
                                  const struct CombinePlan* merge = nullptr);
cudaError_t launch_tree_attn_mma(goose_ctx* c, const __nv_bfloat16* q, const __nv_bfloat16* kc,
                                 const __nv_bfloat16* vc, int64_t kv_rows, const int64_t* row_off, const int32_t* ctx_len,
                                 const int32_t* parent, const int32_t* n_nodes, int S, int B, int H, int Hkv, float scale,
                                 __nv_bfloat16* out, float* lse, cudaStream_t st);
cudaError_t launch_tree_attn_umma(goose_ctx* c, const __nv_bfloat16* q, const __nv_bfloat16* kc,
                                  const __nv_bfloat16* vc, int64_t kv_rows, const int64_t* row_off,
                                  const int32_t* ctx_len, const int32_t* parent, const int32_t* n_nodes, int S, int B, int H,
                                  int Hkv, float scale, __nv_bfloat16* out, float* lse, cudaStream_t st,
                                  struct CombinePlan* defer_merge = nullptr);

cudaError_t launch_bounded_wait_selftest(goose_ctx* c, long long limit_cycles, int32_t* result, cudaStream_t st);

// split count of the mma kernel's fixed grid: ctx_len lives on the device, so it depends only on S, H and the SM count
int mma_splits(const goose_ctx* c, int S, int H);

// per-device kernel attributes (dynamic shared memory limits); called once from goose_create
cudaError_t init_mma_kernel();
cudaError_t init_umma_kernel();
cudaError_t init_topk_kernel();
inline cudaError_t init_kernels(goose_ctx*) {
    cudaError_t e = init_mma_kernel();
    if (e == cudaSuccess) e = init_umma_kernel();
    return e != cudaSuccess ? e : init_topk_kernel();
}

// kernel choice of GOOSE_ATTN_AUTO
int auto_attn_impl(const goose_ctx* c, int S, int B, int H);

}  // namespace goose
