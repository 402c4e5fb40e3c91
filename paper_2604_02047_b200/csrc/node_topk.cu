// Per-node argmax and top-k over bf16 logits (Algorithm 3 step 2; batched top-K harvest of App. C.1).
//
// A row is cut into chunks of 32768 elements; one 1024-thread CTA scans one chunk with 128-bit loads
// held in registers (32 values per thread).  The exact order is carried by 32-bit keys
//     (order-preserving 16-bit image of the bf16 value) << 16 | (0xFFFF - index_in_chunk)
// so "largest key" is "largest value, lowest index on ties", all keys are distinct, and a key carries
// its own index.  Building a key costs several instructions per element, so keys are built only for
// candidates: packed-bf16 maxima give every thread's maximum, redux.sync rounds give the k-th largest
// thread maximum T of the CTA (every top-k element is >= T), and only the elements >= T (about k of
// 32768) are turned into keys and ranked by one warp.  Rows with more than 1024 elements tied at or
// above T (a constant row) take an exact slow path over all keys.  Rows longer than one chunk
// (V > 32768) finish with a merge of the chunks' candidates by the last CTA to arrive for the row
// (arrival counter, no spinning).
#include <mutex>

#include "goose_internal.cuh"

namespace goose {

constexpr int kTopkThreads = 1024;
constexpr int kTopkPerThread = 32;                          // 4 x 128-bit loads
constexpr int kTopkChunk = kTopkThreads * kTopkPerThread;    // 32768 elements
constexpr int kTopkMaxChunks = GOOSE_MAX_V / kTopkChunk;     // 8

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

// 8 consecutive bf16 of a row starting at element idx (a multiple of 8); elements past V read as -inf.
// Plain cached loads: the row chunk is read a second time (from L1/L2) once the threshold is known,
// which keeps the 32 values per thread out of the register file between the two passes.
__device__ __forceinline__ uint4 load8(const unsigned short* rowp, int idx, int V) {
    if (idx + 8 <= V) return __ldg(reinterpret_cast<const uint4*>(rowp + idx));
    unsigned short t[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) t[e] = (idx + e < V) ? rowp[idx + e] : (unsigned short)0xFF80u;
    return make_uint4(t[0] | ((uint32_t)t[1] << 16), t[2] | ((uint32_t)t[3] << 16),
                      t[4] | ((uint32_t)t[5] << 16), t[6] | ((uint32_t)t[7] << 16));
}

__device__ __forceinline__ u64 warp_max_u64(u64 v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        u64 other = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = other > v ? other : v;
    }
    return v;
}

constexpr int kTopkListCap = 1024;                           // candidate list of the fast path

__device__ __forceinline__ uint32_t bits_of_sortable16(uint32_t s) {
    return (s & 0x8000u) ? (s ^ 0x8000u) : (~s & 0xFFFFu);
}
__device__ __forceinline__ __nv_bfloat162 as_bf162(uint32_t w) { return *reinterpret_cast<__nv_bfloat162*>(&w); }
__device__ __forceinline__ uint32_t as_u32(__nv_bfloat162 v) { return *reinterpret_cast<uint32_t*>(&v); }

// LSE = true additionally returns the row's log-sum-exp (for the softmax scores of the harvest): the second
// pass sums exp(x - chunk max) over every element, chunks are merged like split softmax partials.
template <int KCAP, bool LSE>
__global__ void __launch_bounds__(kTopkThreads, 2)
node_topk_kernel(const __nv_bfloat16* __restrict__ logits, int V, int64_t ldl, int k, int chunks,
                 u64* __restrict__ ws_cand, int32_t* __restrict__ row_counters,
                 int32_t* __restrict__ argmax, int32_t* __restrict__ ids, float* __restrict__ vals,
                 float* __restrict__ row_lse, float2* __restrict__ ws_lse) {
    __shared__ float s_sum[32];
    __shared__ uint32_t s_cmax;
    __shared__ uint32_t s_cand[32 * KCAP];               // per-warp winners (thread maxima, or exact keys)
    __shared__ uint32_t s_list[kTopkListCap];            // fast path: keys of all elements >= threshold
    __shared__ u64 s_merge[kTopkMaxChunks * KCAP];
    __shared__ uint32_t s_thresh;
    __shared__ int s_count;
    __shared__ int s_last;

    const int row = blockIdx.y;
    const int chunk = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned short* rowp = reinterpret_cast<const unsigned short*>(logits) + (size_t)row * ldl;
    const int base = chunk * kTopkChunk;
    if (tid == 0) s_count = 0;
    pdl_wait();
    pdl_trigger();

    // ---- phase 1: 32 values per thread (element (it, e) of thread tid sits at chunk offset
    //      it*8192 + tid*8 + e); thread maximum with packed bf16 max
    __nv_bfloat162 m2;
    {
        uint4 v4[4];
#pragma unroll
        for (int it = 0; it < 4; ++it) v4[it] = load8(rowp, base + it * (kTopkThreads * 8) + tid * 8, V);
        m2 = __hmax2(as_bf162(v4[0].x), as_bf162(v4[0].y));
        m2 = __hmax2(m2, __hmax2(as_bf162(v4[0].z), as_bf162(v4[0].w)));
#pragma unroll
        for (int it = 1; it < 4; ++it) {
            m2 = __hmax2(m2, __hmax2(as_bf162(v4[it].x), as_bf162(v4[it].y)));
            m2 = __hmax2(m2, __hmax2(as_bf162(v4[it].z), as_bf162(v4[it].w)));
        }
    }
    const uint32_t mw = as_u32(m2);
    const uint32_t s_lo = sortable16(mw & 0xFFFFu), s_hi = sortable16(mw >> 16);
    uint32_t tmax = s_lo > s_hi ? s_lo : s_hi;

    // ---- phase 2: each warp lists its k largest thread maxima (descending; equal maxima are kept)
    for (int r = 0; r < k; ++r) {
        const uint32_t w = __reduce_max_sync(0xFFFFFFFFu, tmax);
        const uint32_t owners = __ballot_sync(0xFFFFFFFFu, tmax == w);
        if (lane == 0) s_cand[warp * KCAP + r] = w;
        if (lane == __ffs(owners) - 1) tmax = 0;
    }
    __syncthreads();

    // ---- phase 3: warp 0 finds T = the k-th largest thread maximum of the CTA.  At least k elements are
    //      >= T, hence every one of the chunk's k best is >= T.
    if (warp == 0) {
        int ptr = 0;                                     // lane l walks warp l's sorted list
        uint32_t cur = s_cand[lane * KCAP];
        uint32_t w = 0;
        for (int r = 0; r < k; ++r) {
            w = __reduce_max_sync(0xFFFFFFFFu, cur);
            if (LSE && r == 0 && lane == 0) s_cmax = w;   // the chunk's maximum
            const uint32_t owners = __ballot_sync(0xFFFFFFFFu, cur == w);
            if (lane == __ffs(owners) - 1) {
                ++ptr;
                cur = ptr < k ? s_cand[lane * KCAP + ptr] : 0u;
            }
        }
        if (lane == 0) s_thresh = w;
    }
    __syncthreads();

    // ---- phase 4: every element >= T becomes a full key (value image << 16 | 0xFFFF - index in chunk)
    const uint32_t thr_s = s_thresh;
    float esum = 0.f;
    const float cmax = LSE ? __uint_as_float(bits_of_sortable16(s_cmax) << 16) : 0.f;
    {
        const uint32_t tb = bits_of_sortable16(thr_s);
        const __nv_bfloat162 t2 = as_bf162(tb | (tb << 16));
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const uint4 v4 = load8(rowp, base + it * (kTopkThreads * 8) + tid * 8, V);
            const uint32_t wds[4] = {v4.x, v4.y, v4.z, v4.w};
            if (LSE) {                                   // elements past V were loaded as -inf: exp gives 0
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    esum += exp2f((__uint_as_float(wds[q] << 16) - cmax) * 1.4426950408889634f);
                    esum += exp2f((__uint_as_float(wds[q] & 0xFFFF0000u) - cmax) * 1.4426950408889634f);
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t ge = __hge2_mask(as_bf162(wds[q]), t2);
                if (ge) {
                    const int off = it * (kTopkThreads * 8) + tid * 8 + q * 2;
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        if (((ge >> (16 * e)) & 1u) && base + off + e < V) {
                            const uint32_t bits = e ? (wds[q] >> 16) : (wds[q] & 0xFFFFu);
                            const int pos = atomicAdd(&s_count, 1);
                            if (pos < kTopkListCap) s_list[pos] = (sortable16(bits) << 16) | (0xFFFFu - (uint32_t)(off + e));
                        }
                    }
                }
            }
        }
    }
    if (LSE) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) esum += __shfl_xor_sync(0xFFFFFFFFu, esum, o);
        if (lane == 0) s_sum[warp] = esum;
    }
    __syncthreads();
    const int n_list = s_count;
    float csum = 0.f;                                    // warp 0: the chunk's sum of exp(x - cmax)
    if (LSE && warp == 0) {
        csum = s_sum[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(0xFFFFFFFFu, csum, o);
    }

    uint32_t mine = 0;                                   // warp 0: lane r ends up with the r-th winner
    if (n_list <= kTopkListCap) {
        // ---- phase 5 (fast path): warp 0 selects the k best of the list
        if (warp != 0) return;
        for (int r = 0; r < k; ++r) {
            uint32_t m = 0;
            for (int j = lane; j < n_list; j += 32) m = s_list[j] > m ? s_list[j] : m;
            const uint32_t w = __reduce_max_sync(0xFFFFFFFFu, m);
            if (lane == r) mine = w;
            if (w != 0)
                for (int j = lane; j < n_list; j += 32)
                    if (s_list[j] == w) s_list[j] = 0;
            __syncwarp();
        }
    } else {
        // ---- slow path (more than kTopkListCap elements tie at or above T, e.g. a constant row):
        //      exact rounds on full keys of all 32 values per thread
        //      exact rounds on full keys, rebuilt from the (cached) row whenever a lane needs its next best
        // largest key of this thread strictly below `bound` (all keys are distinct)
        auto best_below = [&](uint32_t bound) -> uint32_t {
            uint32_t nb = 0;
#pragma unroll
            for (int it = 0; it < 4; ++it) {
                const int off0 = it * (kTopkThreads * 8) + tid * 8;
                const uint4 v4 = load8(rowp, base + off0, V);
                const uint32_t wds[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const uint32_t bits = (e & 1) ? (wds[e >> 1] >> 16) : (wds[e >> 1] & 0xFFFFu);
                    const uint32_t kk = (base + off0 + e < V) ? ((sortable16(bits) << 16) | (0xFFFFu - (uint32_t)(off0 + e))) : 0u;
                    nb = (kk < bound && kk > nb) ? kk : nb;
                }
            }
            return nb;
        };
        uint32_t best = best_below(0xFFFFFFFFu);
        __syncthreads();                                 // s_cand is reused
        for (int r = 0; r < k; ++r) {
            const uint32_t w = __reduce_max_sync(0xFFFFFFFFu, best);
            if (lane == 0) s_cand[warp * KCAP + r] = w;
            if (best == w && w != 0) best = best_below(w);
        }
        __syncthreads();
        if (warp != 0) return;
        uint32_t c[KCAP];
        uint32_t lm = 0;
#pragma unroll
        for (int j = 0; j < KCAP; ++j) {
            c[j] = (j < k) ? s_cand[lane * KCAP + j] : 0u;
            lm = c[j] > lm ? c[j] : lm;
        }
        for (int r = 0; r < k; ++r) {
            uint32_t w = __reduce_max_sync(0xFFFFFFFFu, lm);
            if (lane == r) mine = w;
            if (lm == w && w != 0) {
                uint32_t nb = 0;
#pragma unroll
                for (int j = 0; j < KCAP; ++j) {
                    c[j] = (c[j] == w) ? 0u : c[j];
                    nb = c[j] > nb ? c[j] : nb;
                }
                lm = nb;
            }
        }
    }
    int32_t my_id = base + (int32_t)(0xFFFFu - (mine & 0xFFFFu));
    uint32_t my_sv = mine >> 16;

    if (chunks > 1) {
        // cross-chunk merge on 64-bit keys (value image << 32 | ~global index)
        u64* dst = ws_cand + ((size_t)row * chunks + chunk) * kMaxK;
        if (lane < k) dst[lane] = mine ? (((u64)my_sv << 32) | (u64)(0xFFFFFFFFu - (uint32_t)my_id)) : 0ull;
        if (LSE && lane == 0) ws_lse[(size_t)row * chunks + chunk] = make_float2(cmax, csum);
        __threadfence();
        __syncwarp();
        if (lane == 0) {
            int old = atomicAdd(&row_counters[row], 1);
            s_last = (old == chunks - 1);
        }
        __syncwarp();
        if (!s_last) return;
        __threadfence();
        const u64* src = ws_cand + (size_t)row * chunks * kMaxK;
        const int n = chunks * k;
        for (int j = lane; j < n; j += 32) s_merge[j] = __ldcg(src + (size_t)(j / k) * kMaxK + (j % k));
        __syncwarp();
        u64 win = 0;
        for (int r = 0; r < k; ++r) {
            u64 m = 0;
            for (int j = lane; j < n; j += 32) m = s_merge[j] > m ? s_merge[j] : m;
            u64 w = warp_max_u64(m);
            if (lane == r) win = w;
            if (w != 0)
                for (int j = lane; j < n; j += 32)
                    if (s_merge[j] == w) s_merge[j] = 0;
            __syncwarp();
        }
        if (lane == 0) row_counters[row] = 0;               // ready for the next launch
        my_id = (int32_t)(0xFFFFFFFFu - (uint32_t)(win & 0xFFFFFFFFull));
        my_sv = (uint32_t)(win >> 32);
        if (LSE && lane == 0) {
            float M = -INFINITY;
            for (int c = 0; c < chunks; ++c) M = fmaxf(M, __ldcg(&ws_lse[(size_t)row * chunks + c]).x);
            float sum = 0.f;
            for (int c = 0; c < chunks; ++c) {
                const float2 ms = __ldcg(&ws_lse[(size_t)row * chunks + c]);
                sum += ms.y * expf(ms.x - M);
            }
            row_lse[row] = M + logf(sum);
        }
    } else if (LSE && lane == 0) {
        row_lse[row] = cmax + logf(csum);
    }
    if (lane < k) {
        ids[(size_t)row * k + lane] = my_id;
        if (vals) vals[(size_t)row * k + lane] = value_of_sortable16(my_sv);
        if (lane == 0) argmax[row] = my_id;
    }
}

cudaError_t launch_node_topk(goose_ctx* c, const __nv_bfloat16* logits, int rows, int V, int64_t ldl, int k,
                             int32_t* argmax, int32_t* ids, float* vals, float* row_lse, cudaStream_t st) {
    if (rows == 0) return cudaSuccess;
    int chunks = (V + kTopkChunk - 1) / kTopkChunk;
    for (int r0 = 0; r0 < rows; r0 += 65535) {               // gridDim.y limit
        int nr = rows - r0 < 65535 ? rows - r0 : 65535;
        dim3 grid(chunks, nr);
        const __nv_bfloat16* lp = logits + (size_t)r0 * ldl;
        u64* ws = c->topk_cand + (size_t)r0 * chunks * kMaxK;
        float* vp = vals ? vals + (size_t)r0 * k : nullptr;
        float* lsep = row_lse ? row_lse + r0 : nullptr;
        float2* wl = reinterpret_cast<float2*>(c->topk_lse_ws) + (size_t)r0 * chunks;
        auto kern = row_lse ? (k <= 8 ? node_topk_kernel<8, true> : node_topk_kernel<16, true>)
                            : (k <= 8 ? node_topk_kernel<8, false> : node_topk_kernel<16, false>);
        cudaError_t e = launch_pdl(kern, grid, dim3(kTopkThreads), 0, st, lp, V, ldl, k, chunks, ws, c->row_counters + r0,
                                   argmax + r0, ids + (size_t)r0 * k, vp, lsep, wl);
        c->launches++;
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
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
    {
        // In host code the name g_static_topk is only a handle for the runtime, not a device address:
        // resolve the address once per device, with that device current.
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_ptr[dev]) {
            u64* p = nullptr;
            if (cudaGetSymbolAddress((void**)&p, g_static_topk) != cudaSuccess || !p) return GOOSE_ECUDA;
            g_static_ptr[dev] = p;
        }
        scratch = g_static_ptr[dev];
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int chunks = (V + kTopkChunk - 1) / kTopkChunk;
    // the counters must start at zero; the array keeps whatever an earlier (possibly interrupted) call left
    int32_t* counters = reinterpret_cast<int32_t*>(scratch + kStaticCandWords);
    if (chunks > 1 && cudaMemsetAsync(counters, 0, sizeof(int32_t) * (size_t)rows, st) != cudaSuccess)
        return GOOSE_ECUDA;
    dim3 grid(chunks, rows);                                             // rows <= 2048 < 65535
    cudaError_t e = launch_pdl(k <= 8 ? node_topk_kernel<8, false> : node_topk_kernel<16, false>, grid, dim3(kTopkThreads), 0,
                               st, static_cast<const __nv_bfloat16*>(logits), V, ldl, k, chunks, scratch, counters, argmax,
                               topk_ids, topk_vals, static_cast<float*>(nullptr), static_cast<float2*>(nullptr));
    return e == cudaSuccess ? GOOSE_OK : GOOSE_ECUDA;
}
