// Per-node argmax and top-k over bf16 logits (Algorithm 3 step 2; batched top-K harvest of App. C.1).
//
// A row is cut into chunks of 32768 elements; the (row, chunk) items, in row-major order, are dealt in contiguous
// ranges to a persistent grid of one 1024-thread CTA per SM.  One thread streams the CTA's items into a ring of
// three 64 KB shared-memory stages with bulk asynchronous copies (cp.async.bulk, mbarrier completion), so HBM keeps
// streaming while the CTA selects; every thread then takes 32 values of the current item into registers.
// The exact order is carried by 32-bit keys
//     (order-preserving 16-bit image of the bf16 value) << 16 | (0xFFFF - index_in_chunk)
// so "largest key" is "largest value, lowest index on ties", all keys are distinct, and a key carries its own
// index.  Building a key costs several instructions per element, so keys are built only for candidates: packed-bf16
// maxima give every thread's maximum, one redux.sync gives every warp's maximum, and T = the k-th largest of the 32
// warp maxima is a threshold with at least k elements at or above it -- hence every one of the chunk's k best is
// >= T.  Only the elements >= T (about ten of 32768) become keys, and one warp ranks them.  Selections among up
// to 32 distinct keys are done by rank counting (every lane counts the keys above its own: independent compares
// instead of k dependent warp-wide reduction rounds).  Chunks with more than
// 1024 elements at or above T (a constant row) take an exact slow path over all keys.  The chunks of a row are merged
// by the CTA as it walks them; a row whose chunks are spread over several CTAs is finished by the last of those CTAs
// to arrive (arrival counter, no spinning).  Every mbarrier wait is bounded: when one runs out the CTA reports
// GOOSE_ST_TIMEOUT, drains its own copies in flight (bounded again) and returns.
#include <mutex>

#include "goose_internal.cuh"

namespace goose {

constexpr int kTopkThreads = 1024;
constexpr int kTopkPerThread = 32;                          // 4 x 128-bit shared-memory loads
constexpr int kTopkChunk = kTopkThreads * kTopkPerThread;    // 32768 elements
constexpr int kTopkMaxChunks = GOOSE_MAX_V / kTopkChunk;     // 8
constexpr int kTopkStages = 3;
constexpr int kTopkStageBytes = kTopkChunk * 2;              // 64 KB
constexpr int kTopkSmem = kTopkStages * kTopkStageBytes;     // dynamic shared memory of the kernel
constexpr long long kTopkWaitCycles = 2000000000ll;          // bound of every wait: about one second of SM clock

typedef unsigned long long u64;

__device__ __forceinline__ uint32_t sortable16(uint32_t bits) {
    bits &= 0xFFFFu;
    if (bits == 0x8000u) bits = 0;                           // -0.0 == +0.0
    return (bits & 0x8000u) ? (~bits & 0xFFFFu) : (bits | 0x8000u);
}

__device__ __forceinline__ float value_of_sortable16(uint32_t s) {
    uint32_t bits = (s & 0x8000u) ? (s ^ 0x8000u) : (~s & 0xFFFFu);
    return __uint_as_float(bits << 16);
}

constexpr int kTopkListCap = 1024;                           // candidate list of the fast path

__device__ __forceinline__ uint32_t bits_of_sortable16(uint32_t s) {
    return (s & 0x8000u) ? (s ^ 0x8000u) : (~s & 0xFFFFu);
}
__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t w) { return *reinterpret_cast<__nv_bfloat162*>(&w); }
__device__ __forceinline__ uint32_t as_u32(__nv_bfloat162 v) { return *reinterpret_cast<uint32_t*>(&v); }

// largest 64-bit key of the warp: two 32-bit redux rounds (high words, then low words among the lanes that tie)
__device__ __forceinline__ u64 warp_max_u64(u64 v) {
    const uint32_t hi = (uint32_t)(v >> 32), lo = (uint32_t)v;
    const uint32_t mh = __reduce_max_sync(0xFFFFFFFFu, hi);
    const uint32_t ml = __reduce_max_sync(0xFFFFFFFFu, hi == mh ? lo : 0u);
    return ((u64)mh << 32) | ml;
}


namespace {
__device__ __forceinline__ uint32_t topk_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
}  // namespace

// LSE = true additionally returns the row's log-sum-exp (for the softmax scores of the harvest): the second
// pass sums exp(x - chunk max) over every element, chunks are merged like split softmax partials.
// COUNTS = false is the instantiation for n_nodes == NULL (the item list is known before the dependency wait)
template <int KCAP, bool LSE, bool COUNTS>
__global__ void __launch_bounds__(kTopkThreads, 1)
node_topk_kernel(const __nv_bfloat16* __restrict__ logits, long long items_all, int V, int64_t ldl, int k, int chunks,
                 u64* __restrict__ ws_cand, int32_t* __restrict__ row_counters,
                 int32_t* __restrict__ argmax, int32_t* __restrict__ ids, float* __restrict__ vals,
                 float* __restrict__ row_lse, float2* __restrict__ ws_lse, int32_t* __restrict__ status,
                 int inputs_ready, const int32_t* __restrict__ n_nodes, int S, int B) {
    extern __shared__ __align__(128) unsigned char s_stage[];   // kTopkStages x 64 KB
    __shared__ u64 s_full[kTopkStages];
    __shared__ float s_sum[32];
    __shared__ __align__(16) uint32_t s_wmax[32];        // warp maxima as distinct keys: value image << 5 | 31 - warp
    __shared__ __align__(16) uint32_t s_sel[32];         // rank-ordered keys of a selection
    __shared__ __align__(16) u64 s_m64[32];              // candidates of a 64-bit merge
    __shared__ u64 s_run[kMaxK];
    __shared__ uint32_t s_thresh, s_cmax;
    __shared__ uint32_t s_cand[32 * KCAP];               // slow path: per-warp winners (exact keys)
    __shared__ __align__(16) uint32_t s_list[kTopkListCap];   // fast path: keys of all elements >= threshold; entries
                                                         // 0..31 are zero between items
    __shared__ u64 s_merge[kTopkMaxChunks * KCAP];
    __shared__ int s_count;                              // length of s_list
    __shared__ int s_last;
    __shared__ volatile int s_abort;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = gridDim.x;
    if (!COUNTS) n_nodes = nullptr;
    long long items = items_all;
    long long w_begin = items * blockIdx.x / G, w_end = items * (blockIdx.x + 1) / G;   // final when !COUNTS
    if (tid == 0) {
        for (int i = 0; i < kTopkStages; ++i)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(topk_smem_u32(&s_full[i])));
        s_count = 0; s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 32) s_list[tid] = 0;
    __syncthreads();
    // inputs_ready: the caller guarantees that the logits were complete before the preceding kernel in the stream
    // started (the whole-step call: that kernel is the attention kernel, which neither reads nor writes them).  The
    // CTA then streams and selects at once and only waits for the preceding kernel before its first write to global
    // memory (outputs, cross-CTA scratch); otherwise it waits here, before its first read.
    bool waited = inputs_ready == 0;
    if (waited) pdl_wait();
    pdl_trigger();
    // Per-sequence node counts (n_nodes != NULL; rows = S * B, row s * B + i belongs to node i of sequence s): rows of
    // nodes that do not exist are left out of the item list, so their logits are never read.  The list then runs over
    // the rows that exist, numbered densely ("row" below; the cross-CTA scratch is indexed by it), and row_of() gives
    // the row in memory.  n_nodes[] is an input like the logits: it may be read ahead of the dependency wait.
    if (COUNTS && n_nodes) {
        long long live = 0;
        for (int s = 0; s < S; ++s) live += nodes_of(n_nodes, s, B);
        items = live * chunks;
        w_begin = items * blockIdx.x / G; w_end = items * (blockIdx.x + 1) / G;
    }
    auto row_of = [&](long long r) -> long long {
        if constexpr (!COUNTS) {
            return r;
        } else {
            if (!n_nodes) return r;
            for (int s = 0; s < S; ++s) {
                const int n = nodes_of(n_nodes, s, B);
                if (r < n) return (long long)s * B + r;
                r -= n;
            }
            return 0;                                    // not reached: r is below the number of live rows
        }
    };
    const int n_local = (int)(w_end - w_begin);

    const unsigned short* lg = reinterpret_cast<const unsigned short*>(logits);
    // thread 0: stream item j of this CTA into stage j % kTopkStages (the copy is rounded up to 16 bytes, which
    // stays inside the row because ldl is a multiple of 8 elements)
    auto issue = [&](int j) {
        const long long w = w_begin + j;
        const long long row = w / chunks;
        const int base = (int)(w - row * chunks) * kTopkChunk;
        const int n_valid = min(kTopkChunk, V - base);
        const uint32_t bytes = ((uint32_t)n_valid * 2u + 15u) & ~15u;
        u64* bar = &s_full[j % kTopkStages];
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(topk_smem_u32(bar)), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(topk_smem_u32(s_stage + (j % kTopkStages) * kTopkStageBytes)),
                       "l"(lg + (size_t)row_of(row) * ldl + base), "r"(bytes), "r"(topk_smem_u32(bar)) : "memory");
    };
    int issued = 0;
    if (tid == 0)
        for (; issued < n_local && issued < kTopkStages; ++issued) issue(issued);

    long long row = w_begin / chunks;
    int chunk = (int)(w_begin - row * chunks);
    // warp 0: the current row's k best over the chunks walked so far (lane r: r-th 64-bit key
    // value image << 32 | ~global index; 0 = none) and its running log-sum-exp parts
    u64 run = 0;
    float run_m = -INFINITY, run_s = 0.f;
    bool part_starts_row = false;
    // the item whose candidate list is complete but not yet ranked (warp 0 ranks it while warp 1 finds the next
    // item's threshold): its row, chunk, chunk maximum, and the slow path's result if that path had to run
    long long pend_row = 0;
    int pend_chunk = -1, pend_j = 0;
    uint32_t pend_cmax_s = 0, pend_mine = 0;
    bool pend_has_mine = false;

    // warp 0: rank the pending item's candidates, merge them into the row's list, write what is complete
    auto finish_pending = [&]() {
        if (!waited) { pdl_wait(); waited = true; }      // warp 0 does every global write of the CTA
        const int n_list = s_count;
        uint32_t mine = pend_mine;                       // lane r: the chunk's r-th winner
        if (!pend_has_mine) {
            if (n_list <= 32) {
                // entries n_list..31 are zero: lane l ranks key l among the (distinct) keys
                const uint32_t c = s_list[lane];
                int rank = 0;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    const uint4 w4 = *reinterpret_cast<const uint4*>(&s_list[i]);
                    rank += (w4.x > c) + (w4.y > c) + (w4.z > c) + (w4.w > c);
                }
                __syncwarp();
                if (c != 0) s_sel[rank] = c;
                __syncwarp();
                mine = lane < min(k, n_list) ? s_sel[lane] : 0u;
            } else {
                for (int r = 0; r < k; ++r) {
                    uint32_t m = 0;
                    for (int i = lane; i < n_list; i += 32) m = s_list[i] > m ? s_list[i] : m;
                    const uint32_t w = __reduce_max_sync(0xFFFFFFFFu, m);
                    if (lane == r) mine = w;
                    if (w != 0)
                        for (int i = lane; i < n_list; i += 32)
                            if (s_list[i] == w) s_list[i] = 0;
                    __syncwarp();
                }
            }
        }
        __syncwarp();
        s_list[lane] = 0;                                // entries 0..31 are zero between items
        if (lane == 0) s_count = 0;

        const int base = pend_chunk * kTopkChunk;
        float csum = 0.f;
        const float cmax = LSE ? __uint_as_float(bits_of_sortable16(pend_cmax_s) << 16) : 0.f;
        if (LSE) {
            csum = s_sum[lane];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(0xFFFFFFFFu, csum, o);
        }
        if (chunks == 1) {                               // the chunk is the row: write it out
            const size_t out_row = (size_t)row_of(pend_row);
            if (lane < k) {
                const int32_t id = (int32_t)(0xFFFFu - (mine & 0xFFFFu));
                ids[out_row * k + lane] = id;
                if (vals) vals[out_row * k + lane] = value_of_sortable16(mine >> 16);
                if (lane == 0) argmax[out_row] = id;
            }
            if (LSE && lane == 0) row_lse[out_row] = cmax + logf(csum);
            return;
        }
        const bool part_begins = (pend_j == 0) || (pend_chunk == 0);
        const bool part_ends = (pend_j == n_local - 1) || (pend_chunk == chunks - 1);
        if (part_begins) part_starts_row = (pend_chunk == 0);
        // this chunk's winners as 64-bit keys of the row
        const u64 ck = mine ? (((u64)(mine >> 16) << 32) | (u64)(0xFFFFFFFFu - (uint32_t)(base + (int)(0xFFFFu - (mine & 0xFFFFu))))) : 0ull;
        if (part_begins) {
            run = lane < k ? ck : 0ull;
            run_m = cmax; run_s = csum;
        } else {
            // merge the running list and the chunk's (k keys each, all distinct): lanes 0..15 offer the running
            // list, lanes 16..31 the chunk's, every lane counts the keys above its own
            const u64 shifted = __shfl_sync(0xFFFFFFFFu, ck, (lane + 16) & 31);   // lane 16 + r <- ck of lane r
            const u64 cand = lane < 16 ? (lane < k ? run : 0ull) : (lane - 16 < k ? shifted : 0ull);
            s_m64[lane] = cand;
            if (lane < kMaxK) s_run[lane] = 0;
            __syncwarp();
            int rank = 0;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const ulonglong2 w2 = *reinterpret_cast<const ulonglong2*>(&s_m64[i]);
                rank += (w2.x > cand) + (w2.y > cand);
            }
            if (cand != 0 && rank < k) s_run[rank] = cand;
            __syncwarp();
            run = lane < k ? s_run[lane] : 0ull;
            __syncwarp();
            if (LSE) {
                const float M = fmaxf(run_m, cmax);
                run_s = run_s * expf(run_m - M) + csum * expf(cmax - M);
                run_m = M;
            }
        }
        if (!part_ends) return;
        u64 win = run;
        float fin_m = run_m, fin_s = run_s;
        if (!(part_starts_row && pend_chunk == chunks - 1)) {
            // the row's chunks are spread over several CTAs: CTAs c_first..c_last each hold one part
            auto cta_of = [&](long long w) -> int {      // the CTA whose range contains item w
                int c = (int)((w * G) / items);
                while (c + 1 < G && items * (c + 1) / G <= w) ++c;
                while (c > 0 && items * c / G > w) --c;
                return c;
            };
            const int c_first = cta_of(pend_row * chunks), c_last = cta_of(pend_row * chunks + chunks - 1);
            const int n_parts = c_last - c_first + 1, slot = (int)blockIdx.x - c_first;
            u64* dst = ws_cand + ((size_t)pend_row * chunks + slot) * kMaxK;
            if (lane < k) dst[lane] = run;
            if (LSE && lane == 0) ws_lse[(size_t)pend_row * chunks + slot] = make_float2(run_m, run_s);
            __threadfence();
            __syncwarp();
            if (lane == 0) {
                const int old = atomicAdd(&row_counters[pend_row], 1);
                s_last = (old == n_parts - 1);
            }
            __syncwarp();
            if (!s_last) return;
            __threadfence();
            const u64* src = ws_cand + (size_t)pend_row * chunks * kMaxK;
            const int n = n_parts * k;
            if (n <= 32) {
                const u64 cand = lane < n ? __ldcg(src + (size_t)(lane / k) * kMaxK + (lane % k)) : 0ull;
                s_m64[lane] = cand;
                if (lane < kMaxK) s_run[lane] = 0;
                __syncwarp();
                int rank = 0;
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const ulonglong2 w2 = *reinterpret_cast<const ulonglong2*>(&s_m64[i]);
                    rank += (w2.x > cand) + (w2.y > cand);
                }
                if (cand != 0 && rank < k) s_run[rank] = cand;
                __syncwarp();
                win = lane < k ? s_run[lane] : 0ull;
                __syncwarp();
            } else {
                for (int i = lane; i < n; i += 32) s_merge[i] = __ldcg(src + (size_t)(i / k) * kMaxK + (i % k));
                __syncwarp();
                win = 0;
                for (int r = 0; r < k; ++r) {
                    u64 m = 0;
                    for (int i = lane; i < n; i += 32) m = s_merge[i] > m ? s_merge[i] : m;
                    const u64 w = warp_max_u64(m);
                    if (lane == r) win = w;
                    if (w != 0)
                        for (int i = lane; i < n; i += 32)
                            if (s_merge[i] == w) s_merge[i] = 0;
                    __syncwarp();
                }
            }
            if (lane == 0) row_counters[pend_row] = 0;   // ready for the next launch
            if (LSE && lane == 0) {
                float M = -INFINITY;
                for (int c = 0; c < n_parts; ++c) M = fmaxf(M, __ldcg(&ws_lse[(size_t)pend_row * chunks + c]).x);
                float sum = 0.f;
                for (int c = 0; c < n_parts; ++c) {
                    const float2 ms = __ldcg(&ws_lse[(size_t)pend_row * chunks + c]);
                    sum += ms.y * expf(ms.x - M);
                }
                fin_m = M; fin_s = sum;
            }
        }
        const size_t out_row = (size_t)row_of(pend_row);
        if (lane < k) {
            const int32_t id = (int32_t)(0xFFFFFFFFu - (uint32_t)(win & 0xFFFFFFFFull));
            ids[out_row * k + lane] = id;
            if (vals) vals[out_row * k + lane] = value_of_sortable16((uint32_t)(win >> 32));
            if (lane == 0) argmax[out_row] = id;
        }
        if (LSE && lane == 0) row_lse[out_row] = fin_m + logf(fin_s);
    };

    for (int j = 0; j < n_local; ++j) {
        const int st = j % kTopkStages;
        const int base = chunk * kTopkChunk;
        const int n_valid = min(kTopkChunk, V - base);
        const unsigned char* sp = s_stage + st * kTopkStageBytes;
        // a wait that runs out raises the CTA's abort flag; everybody learns of it behind the next barrier
        const bool have = mbar_wait_bounded(&s_full[st], (uint32_t)(j / kTopkStages) & 1u, kTopkWaitCycles, &s_abort) == 0;
        if (!have) s_abort = 1;

        // ---- phase 1: 32 values per thread into registers (element (it, e) of thread tid sits at chunk offset
        //      it*8192 + tid*8 + e); elements past the row's end read as -inf; thread maximum with packed bf16 max
        uint32_t x[16];
        if (have) {
#pragma unroll
            for (int it = 0; it < 4; ++it) {
                const uint4 v4 = *reinterpret_cast<const uint4*>(sp + (size_t)(it * (kTopkThreads * 8) + tid * 8) * 2);
                x[4 * it] = v4.x; x[4 * it + 1] = v4.y; x[4 * it + 2] = v4.z; x[4 * it + 3] = v4.w;
            }
            if (n_valid < kTopkChunk) {
#pragma unroll
                for (int it = 0; it < 4; ++it) {
                    const int off0 = it * (kTopkThreads * 8) + tid * 8;
                    if (off0 + 8 > n_valid) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const uint32_t lo = (off0 + 2 * q < n_valid) ? (x[4 * it + q] & 0xFFFFu) : 0xFF80u;
                            const uint32_t hi = (off0 + 2 * q + 1 < n_valid) ? (x[4 * it + q] >> 16) : 0xFF80u;
                            x[4 * it + q] = lo | (hi << 16);
                        }
                    }
                }
            }
        } else {
#pragma unroll
            for (int q = 0; q < 16; ++q) x[q] = 0xFF80FF80u;
        }
        __nv_bfloat162 m2 = __hmax2(as_bf162(x[0]), as_bf162(x[1]));
#pragma unroll
        for (int q = 2; q < 16; q += 2) m2 = __hmax2(m2, __hmax2(as_bf162(x[q]), as_bf162(x[q + 1])));
        const uint32_t mw = as_u32(m2);
        const uint32_t s_lo = sortable16(mw & 0xFFFFu), s_hi = sortable16(mw >> 16);
        const uint32_t tmax = s_lo > s_hi ? s_lo : s_hi;   // this thread's maximum (16-bit value image)
        const uint32_t wmax = __reduce_max_sync(0xFFFFFFFFu, tmax);
        if (lane == 0) s_wmax[warp] = (wmax << 5) | (uint32_t)(31 - warp);
        __syncthreads();
        if (s_abort) {
            // give up as one: report, wait (bounded) for this thread's copies still in flight, return
            if (!waited) pdl_wait();                     // completion of this grid must imply that of the preceding one
            if (tid == 0) {
                if (status) atomicOr(status, GOOSE_ST_TIMEOUT);
                volatile int no_abort = 0;               // draining ignores the abort flag
                for (int jj = j; jj < issued; ++jj)
                    mbar_wait_bounded(&s_full[jj % kTopkStages], (uint32_t)(jj / kTopkStages) & 1u, kTopkWaitCycles, &no_abort);
            }
            return;
        }

        // ---- phase 2, two warps side by side.  Warp 1: T = the k-th largest warp maximum -- lane l counts the warp
        //      maxima above warp l's (the keys are distinct), the lane of rank k-1 holds T.  The k largest warp
        //      maxima are k different elements >= T, hence every one of the chunk's k best is >= T.
        //      Warp 0: ranks the previous item's candidates.
        if (warp == 1) {
            const uint32_t mykey = s_wmax[lane];
            int rank = 0;
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
                const uint4 w4 = *reinterpret_cast<const uint4*>(&s_wmax[i]);
                rank += (w4.x > mykey) + (w4.y > mykey) + (w4.z > mykey) + (w4.w > mykey);
            }
            if (rank == k - 1) s_thresh = mykey >> 5;
            if (rank == 0) s_cmax = mykey >> 5;          // the chunk's maximum
        } else if (warp == 0 && pend_chunk >= 0) {
            finish_pending();
        }
        __syncthreads();
        const uint32_t thr_s = s_thresh, cmax_s = s_cmax;

        // ---- phase 3: every element >= T becomes a full key (value image << 16 | 0xFFFF - index in chunk).
        //      A thread holds such an element exactly when its maximum is >= T (about ten threads of the CTA); the
        //      warp then looks at that thread's 32 elements together, one lane per element, in the stage.
        float esum = 0.f;
        const float cmax = LSE ? __uint_as_float(bits_of_sortable16(cmax_s) << 16) : 0.f;
        if (LSE) {                                       // elements past the row's end are -inf: exp gives 0
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                esum += exp2f((__uint_as_float(x[q] << 16) - cmax) * 1.4426950408889634f);
                esum += exp2f((__uint_as_float(x[q] & 0xFFFF0000u) - cmax) * 1.4426950408889634f);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) esum += __shfl_xor_sync(0xFFFFFFFFu, esum, o);
            if (lane == 0) s_sum[warp] = esum;
        }
        uint32_t holders = __ballot_sync(0xFFFFFFFFu, tmax >= thr_s);
        while (holders) {
            const int src_tid = (warp << 5) + __ffs(holders) - 1;
            holders &= holders - 1;
            const int off = (lane >> 3) * (kTopkThreads * 8) + src_tid * 8 + (lane & 7);
            const uint32_t sv = sortable16(reinterpret_cast<const unsigned short*>(sp)[off]);
            const bool pass = off < n_valid && sv >= thr_s;
            const uint32_t pm = __ballot_sync(0xFFFFFFFFu, pass);
            int pos0 = 0;
            if (lane == 0) pos0 = atomicAdd(&s_count, __popc(pm));
            pos0 = __shfl_sync(0xFFFFFFFFu, pos0, 0);
            if (pass) {
                const int pos = pos0 + __popc(pm & ((1u << lane) - 1u));
                if (pos < kTopkListCap) s_list[pos] = (sv << 16) | (0xFFFFu - (uint32_t)off);
            }
        }
        __syncthreads();
        // every thread is done with the stage: fetch the item three ahead into it
        if (tid == 0 && issued < n_local) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue(issued);
            ++issued;
        }
        pend_row = row; pend_chunk = chunk; pend_j = j; pend_cmax_s = cmax_s;
        pend_has_mine = false; pend_mine = 0;

        if (s_count > kTopkListCap) {
            // ---- slow path (more than kTopkListCap elements tie at or above T, e.g. a constant row): exact rounds
            //      on full keys, rebuilt from the registers whenever a lane needs its next best.
            // largest key of this thread strictly below `bound` (all keys are distinct)
            auto best_below = [&](uint32_t bound) -> uint32_t {
                uint32_t nb = 0;
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const int off = (q >> 2) * (kTopkThreads * 8) + tid * 8 + (q & 3) * 2;
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const uint32_t bits = e ? (x[q] >> 16) : (x[q] & 0xFFFFu);
                        const uint32_t kk = (off + e < n_valid) ? ((sortable16(bits) << 16) | (0xFFFFu - (uint32_t)(off + e))) : 0u;
                        nb = (kk < bound && kk > nb) ? kk : nb;
                    }
                }
                return nb;
            };
            uint32_t best = best_below(0xFFFFFFFFu);
            for (int r = 0; r < k; ++r) {
                const uint32_t w = __reduce_max_sync(0xFFFFFFFFu, best);
                if (lane == 0) s_cand[warp * KCAP + r] = w;
                if (best == w && w != 0) best = best_below(w);
            }
            __syncthreads();
            if (warp == 0) {
                uint32_t c[KCAP];
                uint32_t lm = 0;
#pragma unroll
                for (int i = 0; i < KCAP; ++i) {
                    c[i] = (i < k) ? s_cand[lane * KCAP + i] : 0u;
                    lm = c[i] > lm ? c[i] : lm;
                }
                for (int r = 0; r < k; ++r) {
                    uint32_t w = __reduce_max_sync(0xFFFFFFFFu, lm);
                    if (lane == r) pend_mine = w;
                    if (lm == w && w != 0) {
                        uint32_t nb = 0;
#pragma unroll
                        for (int i = 0; i < KCAP; ++i) {
                            c[i] = (c[i] == w) ? 0u : c[i];
                            nb = c[i] > nb ? c[i] : nb;
                        }
                        lm = nb;
                    }
                }
            }
            pend_has_mine = true;
            __syncthreads();                             // s_cand is reused by the next slow item
        }
        if (++chunk == chunks) { chunk = 0; ++row; }
    }
    if (warp == 0 && pend_chunk >= 0) finish_pending();  // the CTA's last item
    if (!waited) pdl_wait();                             // a CTA without items, or the warps that wrote nothing
}

namespace {
template <int KCAP, bool LSE>
cudaError_t launch_topk_inst(int grid, cudaStream_t st, const __nv_bfloat16* logits, long long items, int V, int64_t ldl,
                             int k, int chunks, u64* ws, int32_t* counters, int32_t* argmax, int32_t* ids, float* vals,
                             float* row_lse, float2* ws_lse, int32_t* status, int inputs_ready, const int32_t* n_nodes, int S,
                             int B) {
    return launch_pdl(n_nodes ? node_topk_kernel<KCAP, LSE, true> : node_topk_kernel<KCAP, LSE, false>, dim3(grid),
                      dim3(kTopkThreads), kTopkSmem, st, logits, items, V, ldl, k,
                      chunks, ws, counters, argmax, ids, vals, row_lse, ws_lse, status, inputs_ready, n_nodes, S, B);
}

cudaError_t launch_topk_any(int num_sms, cudaStream_t st, const __nv_bfloat16* logits, int rows, int V, int64_t ldl, int k,
                            u64* ws, int32_t* counters, int32_t* argmax, int32_t* ids, float* vals, float* row_lse,
                            float2* ws_lse, int32_t* status, int inputs_ready, const int32_t* n_nodes = nullptr, int B = 0) {
    const int S = (n_nodes && B > 0) ? rows / B : 0;
    const int chunks = (V + kTopkChunk - 1) / kTopkChunk;
    const long long items = (long long)rows * chunks;
    // every CTA gets q = ceil(items / SMs) items or one fewer; using the fewest CTAs that q allows loses no time and
    // makes the ranges fall on row boundaries when q is a multiple of the chunks per row (no cross-CTA merges then)
    const long long q = (items + num_sms - 1) / num_sms;
    const int grid = (int)((items + q - 1) / q);
    if (row_lse)
        return k <= 8 ? launch_topk_inst<8, true>(grid, st, logits, items, V, ldl, k, chunks, ws, counters, argmax, ids, vals, row_lse, ws_lse, status, inputs_ready, n_nodes, S, B)
                      : launch_topk_inst<16, true>(grid, st, logits, items, V, ldl, k, chunks, ws, counters, argmax, ids, vals, row_lse, ws_lse, status, inputs_ready, n_nodes, S, B);
    return k <= 8 ? launch_topk_inst<8, false>(grid, st, logits, items, V, ldl, k, chunks, ws, counters, argmax, ids, vals, row_lse, ws_lse, status, inputs_ready, n_nodes, S, B)
                  : launch_topk_inst<16, false>(grid, st, logits, items, V, ldl, k, chunks, ws, counters, argmax, ids, vals, row_lse, ws_lse, status, inputs_ready, n_nodes, S, B);
}
}  // namespace


// per-device kernel attributes: the stage ring needs the opt-in shared-memory size
cudaError_t init_topk_kernel() {
    cudaError_t e = cudaSuccess;
    auto opt_in = [&](const void* fn) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kTopkSmem);
    };
    opt_in((const void*)node_topk_kernel<8, false, false>);  opt_in((const void*)node_topk_kernel<8, false, true>);
    opt_in((const void*)node_topk_kernel<16, false, false>); opt_in((const void*)node_topk_kernel<16, false, true>);
    opt_in((const void*)node_topk_kernel<8, true, false>);   opt_in((const void*)node_topk_kernel<8, true, true>);
    opt_in((const void*)node_topk_kernel<16, true, false>);  opt_in((const void*)node_topk_kernel<16, true, true>);
    return e;
}

cudaError_t launch_node_topk(goose_ctx* c, const __nv_bfloat16* logits, int rows, int V, int64_t ldl, int k,
                             int32_t* argmax, int32_t* ids, float* vals, float* row_lse, cudaStream_t st,
                             bool inputs_ready, const int32_t* n_nodes, int B) {
    if (rows == 0) return cudaSuccess;
    cudaError_t e = launch_topk_any(c->num_sms, st, logits, rows, V, ldl, k, c->topk_cand, c->row_counters, argmax, ids, vals,
                                    row_lse, reinterpret_cast<float2*>(c->topk_lse_ws), c->status, inputs_ready ? 1 : 0,
                                    n_nodes, B);
    c->launches++;
    return e;
}


// ---------------------------------------------------------------------------------------------------
// goose_node_topk_static: the same kernel for callers that are not allowed to allocate device memory
// (a host that pre-plans all device memory and forbids cudaMalloc at run time, or code running where
// the allocator must not be entered).  The cross-chunk scratch lives in a file-scope device array that
// every GPU loading this library carries until the process exits.
constexpr int kStaticMaxRows = GOOSE_STATIC_TOPK_MAX_ROWS;
constexpr size_t kStaticCandWords = (size_t)kStaticMaxRows * kTopkMaxChunks * kMaxK;   // per (row, chunk) winners: 2 MiB
constexpr size_t kStaticCounterWords = kStaticMaxRows / 2;                             // int32 arrival counters: 8 KiB
static __device__ __align__(256) u64 g_static_topk[kStaticCandWords + kStaticCounterWords];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
u64* g_static_ptr[kMaxDevices] = {};                             // device address of g_static_topk, per device
int g_static_sms[kMaxDevices] = {};                              // SM count, per device
}  // namespace

}  // namespace goose

extern "C" int goose_node_topk_static(const void* logits, int rows, int V, int64_t ldl, int k,
                                      int32_t* argmax, int32_t* topk_ids, float* topk_vals, void* stream) {
    using namespace goose;
    if (!logits || !argmax || !topk_ids) return GOOSE_EINVAL;
    if (rows < 0 || rows > kStaticMaxRows) return GOOSE_EINVAL;          // beyond the static scratch
    if (V < 1 || V > GOOSE_MAX_V || ldl < V || (ldl & 7) != 0) return GOOSE_EINVAL;
    if ((reinterpret_cast<uintptr_t>(logits) & 15u) != 0) return GOOSE_EINVAL;
    if (k < 1 || k > GOOSE_MAX_K || k > V) return GOOSE_EINVAL;
    if (rows == 0) return GOOSE_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GOOSE_ECUDA;
    u64* scratch;
    int num_sms;
    {
        // In host code the name g_static_topk is only a handle for the runtime, not a device address:
        // resolve the address once per device, with that device current.
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_ptr[dev]) {
            u64* p = nullptr;
            int sms = 0;
            if (cudaGetSymbolAddress((void**)&p, g_static_topk) != cudaSuccess || !p) return GOOSE_ECUDA;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return GOOSE_ECUDA;
            if (init_topk_kernel() != cudaSuccess) return GOOSE_ECUDA;   // a function attribute, not an allocation
            g_static_sms[dev] = sms;
            g_static_ptr[dev] = p;
        }
        scratch = g_static_ptr[dev];
        num_sms = g_static_sms[dev];
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int chunks = (V + kTopkChunk - 1) / kTopkChunk;
    // the counters must start at zero; the array keeps whatever an earlier (possibly interrupted) call left
    int32_t* counters = reinterpret_cast<int32_t*>(scratch + kStaticCandWords);
    if (chunks > 1 && cudaMemsetAsync(counters, 0, sizeof(int32_t) * (size_t)rows, st) != cudaSuccess)
        return GOOSE_ECUDA;
    cudaError_t e = launch_topk_any(num_sms, st, static_cast<const __nv_bfloat16*>(logits), rows, V, ldl, k, scratch, counters,
                                    argmax, topk_ids, topk_vals, static_cast<float*>(nullptr), static_cast<float2*>(nullptr),
                                    static_cast<int32_t*>(nullptr), 0);
    return e == cudaSuccess ? GOOSE_OK : GOOSE_ECUDA;
}
