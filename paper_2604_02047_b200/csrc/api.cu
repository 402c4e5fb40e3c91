// C ABI of libgoose: context management, argument validation, and the entry points declared in goose.h.
#include <cstdio>
#include <cstring>
#include <new>

#include "goose_internal.cuh"
#include "tree_attn_combine.cuh"

namespace {

thread_local char g_errbuf[512];
thread_local cudaError_t g_last_cuda = cudaSuccess;

int cuda_fail(cudaError_t e) {
    g_last_cuda = e;
    return GOOSE_ECUDA;
}
#define GOOSE_CUDA(call)                         \
    do {                                         \
        cudaError_t e__ = (call);                \
        if (e__ != cudaSuccess) return cuda_fail(e__); \
    } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// new_ctx_len[] may not overlap ctx_len[]: every block of the compaction launch reads ctx_len[s] while one of them
// writes new_ctx_len[s], so an in-place update would let late blocks move rows relative to the new length
bool ctx_arrays_overlap(const int32_t* ctx_len, const int32_t* new_ctx_len, int S) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(ctx_len), b = reinterpret_cast<uintptr_t>(new_ctx_len);
    const uintptr_t n = sizeof(int32_t) * (uintptr_t)(S > 0 ? S : 1);
    return a < b + n && b < a + n;
}

// the context's workspace, kernel attributes and tensor maps belong to c->device: a stream-ordered call made with
// another device current would fail at launch with an opaque CUDA error
bool on_ctx_device(const goose_ctx* c) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == c->device;
}

int check_shape(const goose_ctx* c, int S, int B, int H, int D) {
    if (!c || !on_ctx_device(c)) return GOOSE_EINVAL;
    if (S < 0 || S > c->max_S) return GOOSE_EINVAL;
    if (B < 1 || B > c->max_B || B > GOOSE_MAX_B) return GOOSE_EINVAL;
    if (H < 1 || H > c->max_H) return GOOSE_EINVAL;
    if (D != GOOSE_HEAD_DIM) return GOOSE_EINVAL;
    return GOOSE_OK;
}

constexpr int kTopkChunkElems = 32768;
constexpr int kTopkMaxChunks = GOOSE_MAX_V / kTopkChunkElems;   // 8

}  // namespace

extern "C" {

const char* goose_strerror(int rc) {
    const char* base;
    switch (rc) {
        case GOOSE_OK: base = "ok"; break;
        case GOOSE_EINVAL: base = "invalid argument"; break;
        case GOOSE_ENOMEM: base = "out of memory"; break;
        case GOOSE_ECUDA: base = "CUDA error"; break;
        case GOOSE_ETIMEOUT: base = "device-side wait timed out"; break;
        default: base = "unknown error"; break;
    }
    if (rc == GOOSE_ECUDA)
        snprintf(g_errbuf, sizeof g_errbuf, "%s: %s", base, cudaGetErrorString(g_last_cuda));
    else
        snprintf(g_errbuf, sizeof g_errbuf, "%s", base);
    return g_errbuf;
}

int goose_create(goose_ctx** out, int device, int max_S, int max_B, int max_H, int head_dim) {
    if (!out) return GOOSE_EINVAL;
    *out = nullptr;
    if (max_S < 1 || max_B < 1 || max_B > GOOSE_MAX_B || max_H < 1 || head_dim != GOOSE_HEAD_DIM) return GOOSE_EINVAL;
    GOOSE_CUDA(cudaSetDevice(device));
    goose_ctx* c = new (std::nothrow) goose_ctx();
    if (!c) return GOOSE_ENOMEM;
    memset(c, 0, sizeof *c);
    c->device = device;
    c->max_S = max_S; c->max_B = max_B; c->max_H = max_H;
    c->attn_impl = GOOSE_ATTN_AUTO;
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) { delete c; return cuda_fail(e); }
    c->num_sms = prop.multiProcessorCount;

    // attention partial slots: two per CTA of the persistent kernel, or heads x splits of the split kernel
    long long heads = (long long)max_S * max_H;
    long long slots = 2LL * c->num_sms + 2;
    if (slots < heads) slots = heads;           // at least one slot per head
    if (slots < 4LL * c->num_sms) slots = 4LL * c->num_sms;
    c->n_slots = (int)slots;
    c->topk_rows_cap = max_S * max_B;
    c->topk_cand_cap = (int64_t)c->topk_rows_cap * kTopkMaxChunks * GOOSE_MAX_K;

    bool ok = true;
    cudaError_t setup_err = cudaSuccess;               // a failure that is not an allocation keeps its own code
    ok = ok && cudaMalloc(&c->partials, sizeof(float) * (size_t)c->n_slots * goose::kPartialFloats) == cudaSuccess;
    ok = ok && cudaMalloc(&c->head_counters, sizeof(int32_t) * (size_t)heads) == cudaSuccess;
    ok = ok && cudaMalloc(&c->topk_cand, sizeof(unsigned long long) * (size_t)c->topk_cand_cap) == cudaSuccess;
    ok = ok && cudaMalloc(&c->row_counters, sizeof(int32_t) * (size_t)c->topk_rows_cap) == cudaSuccess;
    ok = ok && cudaMalloc(&c->topk_lse_ws, sizeof(float) * 2 * (size_t)c->topk_rows_cap * kTopkMaxChunks) == cudaSuccess;
    ok = ok && cudaMalloc(&c->status, sizeof(int32_t) * (size_t)max_S) == cudaSuccess;
    ok = ok && cudaMalloc(&c->selftest_word, sizeof(int32_t)) == cudaSuccess;
    if (ok) {
        ok = ok && cudaMemset(c->head_counters, 0, sizeof(int32_t) * (size_t)heads) == cudaSuccess;
        ok = ok && cudaMemset(c->row_counters, 0, sizeof(int32_t) * (size_t)c->topk_rows_cap) == cudaSuccess;
        ok = ok && cudaMemset(c->status, 0, sizeof(int32_t) * (size_t)max_S) == cudaSuccess;
    }
    if (ok) {
        cudaDriverEntryPointQueryResult qres;
        void* fn = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            c->encode_tiled = fn;
        setup_err = goose::init_kernels(c);            // e.g. a device that is not sm_100: no kernel image
        ok = setup_err == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        goose_destroy(c);
        return setup_err != cudaSuccess ? cuda_fail(setup_err) : GOOSE_ENOMEM;
    }
    *out = c;
    return GOOSE_OK;
}

int goose_destroy(goose_ctx* c) {
    if (!c) return GOOSE_EINVAL;
    cudaSetDevice(c->device);
    cudaFree(c->partials); cudaFree(c->head_counters); cudaFree(c->topk_cand);
    cudaFree(c->row_counters); cudaFree(c->topk_lse_ws); cudaFree(c->status); cudaFree(c->selftest_word); cudaFree(c->stage);
    if (c->pin) cudaFreeHost(c->pin);
    if (c->side) cudaStreamDestroy(c->side);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_logits) cudaEventDestroy(c->ev_logits);
    if (c->side_down) cudaStreamDestroy(c->side_down);
    if (c->ev_attn) cudaEventDestroy(c->ev_attn);
    if (c->ev_out) cudaEventDestroy(c->ev_out);
    delete c;
    return GOOSE_OK;
}

int goose_set_attn_impl(goose_ctx* c, int impl) {
    if (!c || impl < GOOSE_ATTN_AUTO || impl > GOOSE_ATTN_UMMA) return GOOSE_EINVAL;
    c->attn_impl = impl;
    return GOOSE_OK;
}

int64_t goose_launch_count(goose_ctx* c) { return c ? c->launches : -1; }

int goose_tree_attn(goose_ctx* c, const void* q, const void* k_cache, const void* v_cache, int64_t kv_rows,
                    const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent, const int32_t* n_nodes,
                    int S, int B, int H, int D, float scale, void* out, float* lse, void* stream) {
    return goose_tree_attn_gqa(c, q, k_cache, v_cache, kv_rows, row_off, ctx_len, parent, n_nodes, S, B, H, H, D, scale, out,
                               lse, stream);
}

int goose_tree_attn_gqa(goose_ctx* c, const void* q, const void* k_cache, const void* v_cache, int64_t kv_rows,
                        const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent, const int32_t* n_nodes,
                        int S, int B, int H, int Hkv, int D, float scale, void* out, float* lse, void* stream) {
    int rc = check_shape(c, S, B, H, D);
    if (rc) return rc;
    if (Hkv < 1 || H % Hkv != 0 || H / Hkv > GOOSE_MAX_GROUP) return GOOSE_EINVAL;
    if (!q || !k_cache || !v_cache || !row_off || !ctx_len || !parent || !out) return GOOSE_EINVAL;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out)) return GOOSE_EINVAL;
    if (kv_rows < 1 || kv_rows > 0x7FFFFFFFLL) return GOOSE_EINVAL;
    if (!(scale > 0.f) || !(scale < 1e30f)) return GOOSE_EINVAL;
    if (S == 0) return GOOSE_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int impl = c->attn_impl;
    if (impl == GOOSE_ATTN_AUTO) impl = goose::auto_attn_impl(c, S, B, H);
    cudaError_t e;
    if (impl == GOOSE_ATTN_UMMA)
        e = goose::launch_tree_attn_umma(c, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k_cache,
                                         (const __nv_bfloat16*)v_cache, kv_rows, row_off, ctx_len, parent, n_nodes, S, B, H,
                                         Hkv, scale, (__nv_bfloat16*)out, lse, st);
    else
        e = goose::launch_tree_attn_mma(c, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k_cache,
                                        (const __nv_bfloat16*)v_cache, kv_rows, row_off, ctx_len, parent, n_nodes, S, B, H,
                                        Hkv, scale, (__nv_bfloat16*)out, lse, st);
    if (e != cudaSuccess) return cuda_fail(e);
    return GOOSE_OK;
}

int goose_node_topk(goose_ctx* c, const void* logits, int rows, int V, int64_t ldl, int k,
                    const int32_t* n_nodes, int B, int32_t* argmax, int32_t* topk_ids, float* topk_vals, void* stream) {
    if (!c || !on_ctx_device(c) || !logits || !argmax || !topk_ids) return GOOSE_EINVAL;
    if (rows < 0 || rows > c->topk_rows_cap) return GOOSE_EINVAL;
    if (n_nodes && (B < 1 || B > GOOSE_MAX_B || rows % B != 0)) return GOOSE_EINVAL;
    if (V < 1 || V > GOOSE_MAX_V || ldl < V || (ldl & 7) != 0 || !aligned16(logits)) return GOOSE_EINVAL;
    if (k < 1 || k > GOOSE_MAX_K || k > V) return GOOSE_EINVAL;
    cudaError_t e = goose::launch_node_topk(c, (const __nv_bfloat16*)logits, rows, V, ldl, k, argmax, topk_ids,
                                            topk_vals, nullptr, static_cast<cudaStream_t>(stream), false, n_nodes, B);
    if (e != cudaSuccess) return cuda_fail(e);
    return GOOSE_OK;
}

int goose_harvest(goose_ctx* c, const void* logits, int rows, int V, int64_t ldl, int k, const int32_t* row_tok,
                  int table_rows, int32_t* adj_ids, float* adj_scores, int32_t* argmax, int32_t* topk_ids,
                  float* topk_vals, float* row_lse, void* stream) {
    if (!c || !on_ctx_device(c) || !logits || !row_tok || !adj_ids || !adj_scores || !argmax || !topk_ids || !topk_vals ||
        !row_lse)
        return GOOSE_EINVAL;
    if (rows < 0 || rows > c->topk_rows_cap || table_rows < 1) return GOOSE_EINVAL;
    if (V < 1 || V > GOOSE_MAX_V || ldl < V || (ldl & 7) != 0 || !aligned16(logits)) return GOOSE_EINVAL;
    if (k < 1 || k > GOOSE_MAX_K || k > V) return GOOSE_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = goose::launch_node_topk(c, (const __nv_bfloat16*)logits, rows, V, ldl, k, argmax, topk_ids,
                                            topk_vals, row_lse, st);
    if (e != cudaSuccess) return cuda_fail(e);
    e = goose::launch_harvest_scatter(c, row_tok, rows, table_rows, k, topk_ids, topk_vals, row_lse, adj_ids,
                                      adj_scores, st);
    if (e != cudaSuccess) return cuda_fail(e);
    return GOOSE_OK;
}

int goose_accept(goose_ctx* c, const int32_t* draft_tok, const int32_t* parent, const int32_t* n_nodes,
                 const int32_t* argmax, int S, int B, int32_t* path, int32_t* accept_len, int32_t* bonus, void* stream) {
    if (!c || !on_ctx_device(c) || !draft_tok || !parent || !argmax || !path || !accept_len || !bonus) return GOOSE_EINVAL;
    if (S < 0 || S > c->max_S || B < 1 || B > c->max_B) return GOOSE_EINVAL;
    cudaError_t e = goose::launch_accept(c, draft_tok, parent, n_nodes, argmax, S, B, path, accept_len, bonus,
                                         static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    return GOOSE_OK;
}

int goose_kv_compact(goose_ctx* c, void* k_cache, void* v_cache, int64_t kv_rows,
                     const int64_t* row_off, const int32_t* ctx_len, const int32_t* path,
                     const int32_t* accept_len, const int32_t* n_nodes, int S, int B, int H, int D,
                     int32_t* new_ctx_len, void* stream) {
    int rc = check_shape(c, S, B, H, D);
    if (rc) return rc;
    if (!k_cache || !v_cache || !row_off || !ctx_len || !path || !accept_len || !new_ctx_len) return GOOSE_EINVAL;
    if (!aligned16(k_cache) || !aligned16(v_cache) || kv_rows < 1) return GOOSE_EINVAL;
    if (ctx_arrays_overlap(ctx_len, new_ctx_len, S)) return GOOSE_EINVAL;
    cudaError_t e = goose::launch_kv_compact(c, (__nv_bfloat16*)k_cache, (__nv_bfloat16*)v_cache, row_off, ctx_len,
                                             path, accept_len, n_nodes, S, B, H, kv_rows, new_ctx_len,
                                             static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    return GOOSE_OK;
}

int goose_verify_step(goose_ctx* c, const void* q, void* k_cache, void* v_cache, int64_t kv_rows,
                      const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent,
                      const int32_t* n_nodes, const int32_t* draft_tok, const void* logits, int64_t ldl,
                      int S, int B, int H, int D, int V, int k, float scale,
                      void* out, float* lse, int32_t* argmax, int32_t* topk_ids, float* topk_vals,
                      int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* new_ctx_len,
                      void* stream) {
    return goose_verify_step_gqa(c, q, k_cache, v_cache, kv_rows, row_off, ctx_len, parent, n_nodes, draft_tok, logits, ldl,
                                 S, B, H, H, D, V, k, scale, out, lse, argmax, topk_ids, topk_vals, path, accept_len, bonus,
                                 new_ctx_len, stream);
}

int goose_verify_step_gqa(goose_ctx* c, const void* q, void* k_cache, void* v_cache, int64_t kv_rows,
                          const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent,
                          const int32_t* n_nodes, const int32_t* draft_tok, const void* logits, int64_t ldl,
                          int S, int B, int H, int Hkv, int D, int V, int k, float scale,
                          void* out, float* lse, int32_t* argmax, int32_t* topk_ids, float* topk_vals,
                          int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* new_ctx_len,
                          void* stream) {
    return goose_verify_step_harvest(c, q, k_cache, v_cache, kv_rows, row_off, ctx_len, parent, n_nodes, draft_tok, logits,
                                     ldl, S, B, H, Hkv, D, V, k, scale, out, lse, argmax, topk_ids, topk_vals, path, accept_len, bonus,
                                     new_ctx_len, nullptr, 0, nullptr, nullptr, stream);
}

}  // extern "C"

namespace {
// The step's launches.  logits_ready (may be NULL): an event the stream has to wait for before the top-k, for callers
// that produce the logits next to the attention kernels (the host-buffer call uploads them on a side stream).
int enqueue_step(goose_ctx* c, const void* q, void* k_cache, void* v_cache, int64_t kv_rows,
                 const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent,
                 const int32_t* n_nodes, const int32_t* draft_tok, const void* logits, int64_t ldl,
                 int S, int B, int H, int Hkv, int D, int V, int k, float scale,
                 void* out, float* lse, int32_t* argmax, int32_t* topk_ids, float* topk_vals,
                 int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* new_ctx_len,
                 float* row_lse, int table_rows, int32_t* adj_ids, float* adj_scores, void* stream,
                 cudaEvent_t logits_ready, cudaEvent_t attn_done = nullptr);
}  // namespace

extern "C" {

int goose_verify_step_harvest(goose_ctx* c, const void* q, void* k_cache, void* v_cache, int64_t kv_rows,
                              const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent,
                              const int32_t* n_nodes, const int32_t* draft_tok, const void* logits, int64_t ldl,
                              int S, int B, int H, int Hkv, int D, int V, int k, float scale,
                              void* out, float* lse, int32_t* argmax, int32_t* topk_ids, float* topk_vals,
                              int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* new_ctx_len,
                              float* row_lse, int table_rows, int32_t* adj_ids, float* adj_scores, void* stream) {
    return enqueue_step(c, q, k_cache, v_cache, kv_rows, row_off, ctx_len, parent, n_nodes, draft_tok, logits, ldl, S, B, H, Hkv, D, V, k,
                        scale, out, lse, argmax, topk_ids, topk_vals, path, accept_len, bonus, new_ctx_len, row_lse, table_rows,
                        adj_ids, adj_scores, stream, nullptr);
}

}  // extern "C"

namespace {
int enqueue_step(goose_ctx* c, const void* q, void* k_cache, void* v_cache, int64_t kv_rows,
                 const int64_t* row_off, const int32_t* ctx_len, const int32_t* parent,
                 const int32_t* n_nodes, const int32_t* draft_tok, const void* logits, int64_t ldl,
                 int S, int B, int H, int Hkv, int D, int V, int k, float scale,
                 void* out, float* lse, int32_t* argmax, int32_t* topk_ids, float* topk_vals,
                 int32_t* path, int32_t* accept_len, int32_t* bonus, int32_t* new_ctx_len,
                 float* row_lse, int table_rows, int32_t* adj_ids, float* adj_scores, void* stream,
                 cudaEvent_t logits_ready, cudaEvent_t attn_done) {
    // validate everything before enqueueing anything
    const bool harvest = row_lse || adj_ids || adj_scores;
    if (harvest && (!row_lse || !adj_ids || !adj_scores || !topk_vals || table_rows < 1)) return GOOSE_EINVAL;
    int rc = check_shape(c, S, B, H, D);
    if (rc) return rc;
    if (Hkv < 1 || H % Hkv != 0 || H / Hkv > GOOSE_MAX_GROUP) return GOOSE_EINVAL;
    if (!q || !k_cache || !v_cache || !row_off || !ctx_len || !parent || !draft_tok || !logits || !out ||
        !argmax || !topk_ids || !path || !accept_len || !bonus || !new_ctx_len)
        return GOOSE_EINVAL;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out) || !aligned16(logits))
        return GOOSE_EINVAL;
    if (V < 1 || V > GOOSE_MAX_V || ldl < V || (ldl & 7) != 0 || k < 1 || k > GOOSE_MAX_K || k > V) return GOOSE_EINVAL;
    if ((long long)S * B > c->topk_rows_cap || kv_rows < 1 || kv_rows > 0x7FFFFFFFLL) return GOOSE_EINVAL;
    if (ctx_arrays_overlap(ctx_len, new_ctx_len, S)) return GOOSE_EINVAL;
    // Attention.  With the tensor-core kernel the merge of its split heads does not get a launch of its own here: it
    // rides in the step's last launch, beside the walk and the compaction, so the top-k starts the moment the main
    // kernel's CTAs leave their SMs (out[] and lse[] are complete when the step is).
    goose::CombinePlan merge_plan;
    merge_plan.valid = false;
    if (!(scale > 0.f) || !(scale < 1e30f)) return GOOSE_EINVAL;
    {
        int impl = c->attn_impl;
        if (impl == GOOSE_ATTN_AUTO) impl = goose::auto_attn_impl(c, S, B, H);
        // attn_done (the host-buffer call): out[] must be complete as early as possible, so that it can travel to the
        // host while the logits are still on their way up -- the attention then keeps the merge as its own kernel
        if (impl == GOOSE_ATTN_UMMA && S > 0 && !attn_done) {
            cudaError_t ea = goose::launch_tree_attn_umma(c, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k_cache,
                                                          (const __nv_bfloat16*)v_cache, kv_rows, row_off, ctx_len, parent,
                                                          n_nodes, S, B, H, Hkv, scale, (__nv_bfloat16*)out, lse,
                                                          static_cast<cudaStream_t>(stream), &merge_plan);
            if (ea != cudaSuccess) return cuda_fail(ea);
        } else {
            rc = goose_tree_attn_gqa(c, q, k_cache, v_cache, kv_rows, row_off, ctx_len, parent, n_nodes, S, B, H, Hkv, D, scale,
                                     out, lse, stream);
            if (rc) return rc;
        }
        if (attn_done) GOOSE_CUDA(cudaEventRecord(attn_done, static_cast<cudaStream_t>(stream)));
    }
    // the logits are an input of the step: complete before the attention kernel above started, which does not touch
    // them -- so the top-k kernel may read them while that kernel is still running.  With a harvest it also
    // returns every row's log-sum-exp (one pass over the logits serves the walk and the table).
    if (S > 0) {
        // (with logits_ready the kernel cannot start before the event, so reading ahead of its own wait stays safe)
        if (logits_ready) GOOSE_CUDA(cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), logits_ready, 0));
        cudaError_t et = goose::launch_node_topk(c, (const __nv_bfloat16*)logits, S * B, V, ldl, k, argmax, topk_ids, topk_vals,
                                                 harvest ? row_lse : nullptr, static_cast<cudaStream_t>(stream),
                                                 /*inputs_ready=*/true, n_nodes, B);
        if (et != cudaSuccess) return cuda_fail(et);
    }
    // acceptance walk + compaction in one launch (same results as goose_accept followed by goose_kv_compact); with a
    // harvest the launch also carries the table scatter: every logits row predicts the successor of its node's own draft
    // token (padding nodes carry negative tokens and are skipped)
    cudaError_t e = goose::launch_accept_compact(c, (__nv_bfloat16*)k_cache, (__nv_bfloat16*)v_cache, row_off, ctx_len,
                                                 draft_tok, parent, n_nodes, argmax, S, B, Hkv, kv_rows, path, accept_len, bonus,
                                                 new_ctx_len, static_cast<cudaStream_t>(stream), table_rows, k, topk_ids,
                                                 topk_vals, row_lse, harvest ? adj_ids : nullptr, adj_scores, &merge_plan);
    if (e != cudaSuccess) return cuda_fail(e);
    return GOOSE_OK;
}
}  // namespace

extern "C" {

int goose_verify_step_host(goose_ctx* c, void* k_cache, void* v_cache, int64_t kv_rows,
                           const void* h_q, const void* h_k_new, const void* h_v_new,
                           const int64_t* h_row_off, const int32_t* h_ctx_len,
                           const int32_t* h_parent, const int32_t* h_n_nodes, const int32_t* h_draft_tok, const void* h_logits,
                           int S, int B, int H, int D, int V, int k, float scale,
                           void* h_out, int32_t* h_argmax, int32_t* h_topk_ids, float* h_topk_vals,
                           int32_t* h_path, int32_t* h_accept_len, int32_t* h_bonus,
                           int32_t* h_new_ctx_len, void* stream) {
    return goose_verify_step_host_gqa(c, k_cache, v_cache, kv_rows, h_q, h_k_new, h_v_new, h_row_off, h_ctx_len, h_parent,
                                      h_n_nodes, h_draft_tok, h_logits, S, B, H, H, D, V, k, scale, h_out, h_argmax, h_topk_ids,
                                      h_topk_vals, h_path, h_accept_len, h_bonus, h_new_ctx_len, stream);
}

int goose_verify_step_host_gqa(goose_ctx* c, void* k_cache, void* v_cache, int64_t kv_rows,
                               const void* h_q, const void* h_k_new, const void* h_v_new,
                               const int64_t* h_row_off, const int32_t* h_ctx_len,
                               const int32_t* h_parent, const int32_t* h_n_nodes, const int32_t* h_draft_tok,
                               const void* h_logits, int S, int B, int H, int Hkv, int D, int V, int k, float scale,
                               void* h_out, int32_t* h_argmax, int32_t* h_topk_ids, float* h_topk_vals,
                               int32_t* h_path, int32_t* h_accept_len, int32_t* h_bonus,
                               int32_t* h_new_ctx_len, void* stream) {
    if (!c) return GOOSE_EINVAL;
    GOOSE_CUDA(cudaSetDevice(c->device));               // this call selects the context's device itself
    int rc = check_shape(c, S, B, H, D);
    if (rc) return rc;
    if (Hkv < 1 || H % Hkv != 0 || H / Hkv > GOOSE_MAX_GROUP) return GOOSE_EINVAL;
    if (!k_cache || !v_cache || !h_q || !h_k_new || !h_v_new || !h_row_off || !h_ctx_len || !h_parent ||
        !h_draft_tok || !h_logits || !h_out || !h_argmax || !h_topk_ids || !h_path || !h_accept_len || !h_bonus ||
        !h_new_ctx_len)
        return GOOSE_EINVAL;
    if (V < 1 || V > GOOSE_MAX_V || (V & 7) != 0 || k < 1 || k > GOOSE_MAX_K || k > V) return GOOSE_EINVAL;
    if (S == 0) return GOOSE_OK;
    for (int s = 0; s < S; ++s) {
        const int nn = h_n_nodes ? h_n_nodes[s] : B;        // host data: validated here, before anything is enqueued
        if (nn < 0 || nn > B) return GOOSE_EINVAL;
        if (nn > 0 && (h_row_off[s] < 0 || h_ctx_len[s] < 0 || h_row_off[s] + h_ctx_len[s] + nn > kv_rows)) return GOOSE_EINVAL;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // staging layout (256-byte aligned pieces)
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t n_q = (size_t)S * B * H * D * 2, rows = (size_t)S * B;
    size_t off = 0;
    const size_t o_q = off; off = up(off + n_q);
    const size_t o_out = off; off = up(off + n_q);
    const size_t o_logits = off; off = up(off + rows * V * 2);
    const size_t o_rowoff = off; off = up(off + S * 8);
    const size_t o_ctx = off; off = up(off + S * 4);
    const size_t o_parent = off; off = up(off + rows * 4);
    const size_t o_tok = off; off = up(off + rows * 4);
    const size_t o_nn = off; off = up(off + S * 4);
    const size_t o_argmax = off; off = up(off + rows * 4);
    const size_t o_ids = off; off = up(off + rows * k * 4);
    const size_t o_vals = off; off = up(off + rows * k * 4);
    const size_t o_path = off; off = up(off + rows * 4);
    const size_t o_alen = off; off = up(off + S * 4);
    const size_t o_bonus = off; off = up(off + S * 4);
    const size_t o_newctx = off; off = up(off + S * 4);
    if (off > c->stage_bytes) {
        GOOSE_CUDA(cudaStreamSynchronize(st));
        if (c->stage) cudaFree(c->stage);
        c->stage = nullptr; c->stage_bytes = 0;
        if (cudaMalloc(&c->stage, off) != cudaSuccess) { cudaGetLastError(); return GOOSE_ENOMEM; }
        c->stage_bytes = off;
    }
    char* d = static_cast<char*>(c->stage);
    // one-off per context: the side stream and its events, and the pinned block for the small arrays
    if (!c->side) {
        GOOSE_CUDA(cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking));
        GOOSE_CUDA(cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming));
        GOOSE_CUDA(cudaEventCreateWithFlags(&c->ev_logits, cudaEventDisableTiming));
        GOOSE_CUDA(cudaStreamCreateWithFlags(&c->side_down, cudaStreamNonBlocking));
        GOOSE_CUDA(cudaEventCreateWithFlags(&c->ev_attn, cudaEventDisableTiming));
        GOOSE_CUDA(cudaEventCreateWithFlags(&c->ev_out, cudaEventDisableTiming));
    }
    const size_t in_bytes = o_nn + (size_t)S * 4 - o_rowoff;       // row_off | ctx_len | parent | draft_tok | n_nodes (padded as above)
    const size_t out_bytes = o_newctx + (size_t)S * 4 - o_argmax;  // argmax | ids | vals | path | accept_len | bonus | new_ctx
    const size_t pin_need = up(in_bytes) + out_bytes;
    if (pin_need > c->pin_bytes) {
        GOOSE_CUDA(cudaStreamSynchronize(st));
        if (c->pin) cudaFreeHost(c->pin);
        c->pin = nullptr; c->pin_bytes = 0;
        if (cudaHostAlloc(&c->pin, pin_need, cudaHostAllocDefault) != cudaSuccess) { cudaGetLastError(); return GOOSE_ENOMEM; }
        c->pin_bytes = pin_need;
    }
    char* pin_in = static_cast<char*>(c->pin);
    char* pin_out = pin_in + up(in_bytes);
    const size_t row_bytes = (size_t)Hkv * D * 2;       // one cache row

    // what the attention needs first: the small arrays (one copy through the pinned block), Q and the tree rows of K/V
    memcpy(pin_in + (o_rowoff - o_rowoff), h_row_off, (size_t)S * 8);
    memcpy(pin_in + (o_ctx - o_rowoff), h_ctx_len, (size_t)S * 4);
    memcpy(pin_in + (o_parent - o_rowoff), h_parent, rows * 4);
    memcpy(pin_in + (o_tok - o_rowoff), h_draft_tok, rows * 4);
    if (h_n_nodes) memcpy(pin_in + (o_nn - o_rowoff), h_n_nodes, (size_t)S * 4);
    GOOSE_CUDA(cudaMemcpyAsync(d + o_rowoff, pin_in, in_bytes, cudaMemcpyHostToDevice, st));
    GOOSE_CUDA(cudaMemcpyAsync(d + o_q, h_q, n_q, cudaMemcpyHostToDevice, st));
    for (int s = 0; s < S; ++s) {
        const int nn = h_n_nodes ? h_n_nodes[s] : B;        // only the rows of nodes that exist travel
        if (nn == 0) continue;
        size_t dst = (size_t)(h_row_off[s] + h_ctx_len[s]) * row_bytes;
        GOOSE_CUDA(cudaMemcpyAsync((char*)k_cache + dst, (const char*)h_k_new + (size_t)s * B * row_bytes,
                                   (size_t)nn * row_bytes, cudaMemcpyHostToDevice, st));
        GOOSE_CUDA(cudaMemcpyAsync((char*)v_cache + dst, (const char*)h_v_new + (size_t)s * B * row_bytes,
                                   (size_t)nn * row_bytes, cudaMemcpyHostToDevice, st));
    }
    // the logits (most of the bytes, needed by the top-k only) go up on the side stream while the attention kernels run;
    // the fork sits behind the copies above, so they have the host link to themselves and the attention starts first
    GOOSE_CUDA(cudaEventRecord(c->ev_fork, st));
    GOOSE_CUDA(cudaStreamWaitEvent(c->side, c->ev_fork, 0));
    GOOSE_CUDA(cudaMemcpyAsync(d + o_logits, h_logits, rows * V * 2, cudaMemcpyHostToDevice, c->side));
    GOOSE_CUDA(cudaEventRecord(c->ev_logits, c->side));
    rc = enqueue_step(c, d + o_q, k_cache, v_cache, kv_rows, (const int64_t*)(d + o_rowoff),
                      (const int32_t*)(d + o_ctx), (const int32_t*)(d + o_parent),
                      h_n_nodes ? (const int32_t*)(d + o_nn) : nullptr, (const int32_t*)(d + o_tok),
                      d + o_logits, V, S, B, H, Hkv, D, V, k, scale, d + o_out, nullptr, (int32_t*)(d + o_argmax),
                      (int32_t*)(d + o_ids), (float*)(d + o_vals), (int32_t*)(d + o_path),
                      (int32_t*)(d + o_alen), (int32_t*)(d + o_bonus), (int32_t*)(d + o_newctx), nullptr, 0, nullptr, nullptr,
                      stream, c->ev_logits, c->ev_attn);
    if (rc) {
        cudaStreamSynchronize(c->side);                  // nothing of this call may stay in flight behind an error
        return rc;
    }
    // the attention output goes down on its own stream as soon as the attention is done: the link carries it while the
    // logits are still going up the other way
    GOOSE_CUDA(cudaStreamWaitEvent(c->side_down, c->ev_attn, 0));
    GOOSE_CUDA(cudaMemcpyAsync(h_out, d + o_out, n_q, cudaMemcpyDeviceToHost, c->side_down));
    GOOSE_CUDA(cudaEventRecord(c->ev_out, c->side_down));
    GOOSE_CUDA(cudaMemcpyAsync(pin_out, d + o_argmax, out_bytes, cudaMemcpyDeviceToHost, st));   // the small results: one copy
    GOOSE_CUDA(cudaStreamWaitEvent(st, c->ev_out, 0));
    GOOSE_CUDA(cudaStreamSynchronize(st));
    memcpy(h_argmax, pin_out + (o_argmax - o_argmax), rows * 4);
    memcpy(h_topk_ids, pin_out + (o_ids - o_argmax), rows * k * 4);
    if (h_topk_vals) memcpy(h_topk_vals, pin_out + (o_vals - o_argmax), rows * k * 4);
    memcpy(h_path, pin_out + (o_path - o_argmax), rows * 4);
    memcpy(h_accept_len, pin_out + (o_alen - o_argmax), (size_t)S * 4);
    memcpy(h_bonus, pin_out + (o_bonus - o_argmax), (size_t)S * 4);
    memcpy(h_new_ctx_len, pin_out + (o_newctx - o_argmax), (size_t)S * 4);
    return GOOSE_OK;
}

int goose_selftest_bounded_wait(goose_ctx* c, int64_t limit_cycles, void* stream) {
    if (!c || limit_cycles < 1 || limit_cycles > 4000000000LL) return GOOSE_EINVAL;
    GOOSE_CUDA(cudaSetDevice(c->device));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t* d_result = c->selftest_word;
    GOOSE_CUDA(goose::launch_bounded_wait_selftest(c, limit_cycles, d_result, st));
    int32_t h_result = -1;
    GOOSE_CUDA(cudaMemcpyAsync(&h_result, d_result, sizeof h_result, cudaMemcpyDeviceToHost, st));
    GOOSE_CUDA(cudaStreamSynchronize(st));
    return h_result == 0 ? GOOSE_OK : GOOSE_ECUDA;
}

int goose_last_status(goose_ctx* c, int32_t* host_status, int S) {
    if (!c || !host_status || S < 0 || S > c->max_S) return GOOSE_EINVAL;
    GOOSE_CUDA(cudaSetDevice(c->device));
    GOOSE_CUDA(cudaDeviceSynchronize());
    GOOSE_CUDA(cudaMemcpy(host_status, c->status, sizeof(int32_t) * (size_t)S, cudaMemcpyDeviceToHost));
    GOOSE_CUDA(cudaMemset(c->status, 0, sizeof(int32_t) * (size_t)c->max_S));
    int rc = GOOSE_OK;
    for (int s = 0; s < S; ++s)
        if (host_status[s] & GOOSE_ST_TIMEOUT) rc = GOOSE_ETIMEOUT;
    if (rc == GOOSE_ETIMEOUT) {
        // a CTA that gave up never arrived at its row's / head's counter, and the CTAs that had arrived left it non-zero
        // (only the last arriver resets it): clear them all, the device is idle here
        GOOSE_CUDA(cudaMemset(c->head_counters, 0, sizeof(int32_t) * (size_t)c->max_S * (size_t)c->max_H));
        GOOSE_CUDA(cudaMemset(c->row_counters, 0, sizeof(int32_t) * (size_t)c->topk_rows_cap));
    }
    return rc;
}

}  // extern "C"
