// Per-node argmax and top-k over bf16 logits (Algorithm 3 step 2; batched top-K harvest of App. C.1).
//
// A row is cut into chunks of 32768 elements; one 1024-thread CTA scans one chunk with 128-bit loads
// held in registers (32 values per thread).  Inside a chunk every element is a 32-bit key
//     (order-preserving 16-bit image of the bf16 value) << 16 | (0xFFFF - index_in_chunk)
// so "largest key" is "largest value, lowest index on ties", all keys are distinct, and a key carries
// its own index.  Warp-wide maxima are single redux.sync instructions: each warp extracts its k best
// in k rounds (only the lane that owned the winner rescans its registers), warp 0 then selects the
// chunk's k best from the 32*k candidates.  Rows longer than one chunk (V > 32768) finish with a merge
// of the chunks' candidates by the last CTA to arrive for the row (arrival counter, no spinning).
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

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ u64 warp_max_u64(u64 v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        u64 other = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = other > v ? other : v;
    }
    return v;
}

template <int KCAP>
__global__ void __launch_bounds__(kTopkThreads, 1)
node_topk_kernel(const __nv_bfloat16* __restrict__ logits, int V, int64_t ldl, int k, int chunks,
                 u64* __restrict__ ws_cand, int32_t* __restrict__ row_counters,
                 int32_t* __restrict__ argmax, int32_t* __restrict__ ids, float* __restrict__ vals) {
    __shared__ uint32_t s_cand[32 * KCAP];
    __shared__ u64 s_merge[kTopkMaxChunks * KCAP];
    __shared__ int s_last;

    const int row = blockIdx.y;
    const int chunk = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned short* rowp = reinterpret_cast<const unsigned short*>(logits) + (size_t)row * ldl;
    const int base = chunk * kTopkChunk;

    // ---- 32 values per thread: element (it, e) of thread tid sits at chunk offset it*8192 + tid*8 + e
    uint4 raw[4];
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        int idx = base + it * (kTopkThreads * 8) + tid * 8;
        if (idx + 8 <= V) {
            raw[it] = ldg_stream(reinterpret_cast<const uint4*>(rowp + idx));
        } else {
            unsigned short t[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) t[e] = (idx + e < V) ? rowp[idx + e] : (unsigned short)0;
            raw[it].x = t[0] | ((uint32_t)t[1] << 16); raw[it].y = t[2] | ((uint32_t)t[3] << 16);
            raw[it].z = t[4] | ((uint32_t)t[5] << 16); raw[it].w = t[6] | ((uint32_t)t[7] << 16);
        }
    }
    uint32_t key[kTopkPerThread];
    uint32_t best = 0;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        int off = it * (kTopkThreads * 8) + tid * 8;
        uint32_t w[4] = {raw[it].x, raw[it].y, raw[it].z, raw[it].w};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            uint32_t bits = (e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu);
            uint32_t kk = (base + off + e < V) ? ((sortable16(bits) << 16) | (0xFFFFu - (uint32_t)(off + e))) : 0u;
            key[it * 8 + e] = kk;
            best = kk > best ? kk : best;
        }
    }

    // ---- each warp extracts its k best (redux.sync max; the owning lane drops the winner and rescans)
    for (int r = 0; r < k; ++r) {
        uint32_t w = __reduce_max_sync(0xFFFFFFFFu, best);
        if (lane == 0) s_cand[warp * KCAP + r] = w;
        if (best == w && w != 0) {
            uint32_t nb = 0;
#pragma unroll
            for (int j = 0; j < kTopkPerThread; ++j) {
                key[j] = (key[j] == w) ? 0u : key[j];
                nb = key[j] > nb ? key[j] : nb;
            }
            best = nb;
        }
    }
    __syncthreads();
    if (warp != 0) return;

    // ---- warp 0: the chunk's k best out of 32 warps x k candidates (one warp's list per lane)
    uint32_t c[KCAP];
    uint32_t lm = 0;
#pragma unroll
    for (int j = 0; j < KCAP; ++j) {
        c[j] = (j < k) ? s_cand[lane * KCAP + j] : 0u;       // sorted descending within a lane
        lm = c[j] > lm ? c[j] : lm;
    }
    uint32_t mine = 0;                                       // lane r keeps the r-th winner
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
    int32_t my_id = base + (int32_t)(0xFFFFu - (mine & 0xFFFFu));
    uint32_t my_sv = mine >> 16;

    if (chunks > 1) {
        // cross-chunk merge on 64-bit keys (value image << 32 | ~global index)
        u64* dst = ws_cand + ((size_t)row * chunks + chunk) * kMaxK;
        if (lane < k) dst[lane] = mine ? (((u64)my_sv << 32) | (u64)(0xFFFFFFFFu - (uint32_t)my_id)) : 0ull;
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
    }
    if (lane < k) {
        ids[(size_t)row * k + lane] = my_id;
        if (vals) vals[(size_t)row * k + lane] = value_of_sortable16(my_sv);
        if (lane == 0) argmax[row] = my_id;
    }
}

cudaError_t launch_node_topk(goose_ctx* c, const __nv_bfloat16* logits, int rows, int V, int64_t ldl, int k,
                             int32_t* argmax, int32_t* ids, float* vals, cudaStream_t st) {
    if (rows == 0) return cudaSuccess;
    int chunks = (V + kTopkChunk - 1) / kTopkChunk;
    for (int r0 = 0; r0 < rows; r0 += 65535) {               // gridDim.y limit
        int nr = rows - r0 < 65535 ? rows - r0 : 65535;
        dim3 grid(chunks, nr);
        const __nv_bfloat16* lp = logits + (size_t)r0 * ldl;
        u64* ws = c->topk_cand + (size_t)r0 * chunks * kMaxK;
        float* vp = vals ? vals + (size_t)r0 * k : nullptr;
        if (k <= 8)
            node_topk_kernel<8><<<grid, kTopkThreads, 0, st>>>(lp, V, ldl, k, chunks, ws, c->row_counters + r0,
                                                              argmax + r0, ids + (size_t)r0 * k, vp);
        else
            node_topk_kernel<16><<<grid, kTopkThreads, 0, st>>>(lp, V, ldl, k, chunks, ws, c->row_counters + r0,
                                                               argmax + r0, ids + (size_t)r0 * k, vp);
        c->launches++;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace goose
