// Per-node argmax and top-k over bf16 logits (Algorithm 3 step 2; batched top-K harvest of App. C.1).
//
// Every element becomes a 64-bit key  (order-preserving 16-bit image of the bf16 value) << 32 | ~index,
// so "largest key" is "largest value, lowest index on ties" and all keys of a row are distinct.
// A row is cut into chunks of 8192 elements; one CTA scans one chunk with 128-bit loads held in
// registers (32 values per thread), each warp extracts its k best by k rounds of shuffle-max, warp 0
// merges the warps' candidates, and the last CTA to finish a row (arrival counter, no spinning)
// merges the chunks' candidates and writes argmax / ids / values.
#include "goose_internal.cuh"

namespace goose {

constexpr int kTopkThreads = 256;
constexpr int kTopkPerThread = 32;                       // 4 x 128-bit loads
constexpr int kTopkChunk = kTopkThreads * kTopkPerThread;  // 8192 elements
constexpr int kTopkMaxCand = 512;                        // chunks * k limit of the row merge

typedef unsigned long long u64;

__device__ __forceinline__ uint32_t sortable16(uint32_t bits) {
    bits &= 0xFFFFu;
    if (bits == 0x8000u) bits = 0;                       // -0.0 == +0.0
    return (bits & 0x8000u) ? (~bits & 0xFFFFu) : (bits | 0x8000u);
}

__device__ __forceinline__ float value_of_sortable16(uint32_t s) {
    uint32_t bits = (s & 0x8000u) ? (s ^ 0x8000u) : (~s & 0xFFFFu);
    return __uint_as_float(bits << 16);
}

__device__ __forceinline__ u64 warp_max_u64(u64 v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        u64 other = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = other > v ? other : v;
    }
    return v;
}

// k rounds of arg-max over n candidate keys in shared memory (destroys them); one warp.
__device__ __forceinline__ void warp_select(u64* cand, int n, int k, u64* out, int lane) {
    for (int r = 0; r < k; ++r) {
        u64 c = 0;
        for (int j = lane; j < n; j += 32) c = cand[j] > c ? cand[j] : c;
        u64 w = warp_max_u64(c);
        if (lane == 0) out[r] = w;
        if (w != 0)
            for (int j = lane; j < n; j += 32)
                if (cand[j] == w) cand[j] = 0;
        __syncwarp();
    }
}

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__global__ void __launch_bounds__(kTopkThreads)
node_topk_kernel(const __nv_bfloat16* __restrict__ logits, int V, int64_t ldl, int k, int chunks,
                 u64* __restrict__ ws_cand, int32_t* __restrict__ row_counters,
                 int32_t* __restrict__ argmax, int32_t* __restrict__ ids, float* __restrict__ vals) {
    __shared__ u64 s_cand[kTopkMaxCand];
    __shared__ u64 s_out[kMaxK];
    __shared__ int s_last;

    const int row = blockIdx.y;
    const int chunk = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned short* rowp = reinterpret_cast<const unsigned short*>(logits) + (size_t)row * ldl;
    const int base = chunk * kTopkChunk;

    // ---- load 32 values per thread; local key = sortable16 << 16 | (0xFFFF - slot)
    uint32_t key[kTopkPerThread];
    uint4 raw[4];
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        int idx = base + it * (kTopkThreads * 8) + tid * 8;
        if (idx + 8 <= V) {
            raw[it] = ldg_stream(reinterpret_cast<const uint4*>(rowp + idx));
        } else {
            unsigned short t[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) t[e] = (idx + e < V) ? rowp[idx + e] : (unsigned short)0xFFFFu;
            raw[it].x = t[0] | ((uint32_t)t[1] << 16); raw[it].y = t[2] | ((uint32_t)t[3] << 16);
            raw[it].z = t[4] | ((uint32_t)t[5] << 16); raw[it].w = t[6] | ((uint32_t)t[7] << 16);
        }
    }
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        int idx = base + it * (kTopkThreads * 8) + tid * 8;
        uint32_t w[4] = {raw[it].x, raw[it].y, raw[it].z, raw[it].w};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            uint32_t bits = (e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xFFFFu);
            int slot = it * 8 + e;
            key[slot] = (idx + e < V) ? ((sortable16(bits) << 16) | (0xFFFFu - slot)) : 0u;
        }
    }

    // ---- each warp extracts its k best
    uint32_t best = 0;
#pragma unroll
    for (int j = 0; j < kTopkPerThread; ++j) best = key[j] > best ? key[j] : best;
    for (int r = 0; r < k; ++r) {
        u64 c = 0;
        if (best != 0) {
            int slot = 0xFFFF - (int)(best & 0xFFFFu);
            int gidx = base + (slot >> 3) * (kTopkThreads * 8) + tid * 8 + (slot & 7);
            c = ((u64)(best >> 16) << 32) | (u64)(0xFFFFFFFFu - (uint32_t)gidx);
        }
        u64 w = warp_max_u64(c);
        if (lane == 0) s_cand[warp * k + r] = w;
        if (c == w && c != 0) {                         // this lane owned the winner: drop it, rescan
            uint32_t nb = 0;
#pragma unroll
            for (int j = 0; j < kTopkPerThread; ++j) {
                key[j] = (key[j] == best) ? 0u : key[j];
                nb = key[j] > nb ? key[j] : nb;
            }
            best = nb;
        }
    }
    __syncthreads();

    // ---- warp 0 merges the warps' candidates, then (last CTA of the row) the chunks' candidates
    if (warp == 0) {
        warp_select(s_cand, (kTopkThreads / 32) * k, k, s_out, lane);
        int last = 1;
        if (chunks > 1) {
            u64* dst = ws_cand + ((size_t)row * chunks + chunk) * kMaxK;
            if (lane < k) dst[lane] = s_out[lane];
            __threadfence();
            __syncwarp();
            if (lane == 0) {
                int old = atomicAdd(&row_counters[row], 1);
                s_last = (old == chunks - 1);
            }
            __syncwarp();
            last = s_last;
            if (last) {
                __threadfence();
                const u64* src = ws_cand + (size_t)row * chunks * kMaxK;
                for (int j = lane; j < chunks * k; j += 32)
                    s_cand[j] = __ldcg(src + (size_t)(j / k) * kMaxK + (j % k));
                __syncwarp();
                warp_select(s_cand, chunks * k, k, s_out, lane);
                if (lane == 0) row_counters[row] = 0;   // ready for the next launch
            }
        }
        if (last && lane < k) {
            u64 w = s_out[lane];
            int32_t id = (int32_t)(0xFFFFFFFFu - (uint32_t)(w & 0xFFFFFFFFull));
            ids[(size_t)row * k + lane] = id;
            if (vals) vals[(size_t)row * k + lane] = value_of_sortable16((uint32_t)(w >> 32));
            if (lane == 0) argmax[row] = id;
        }
    }
}

cudaError_t launch_node_topk(goose_ctx* c, const __nv_bfloat16* logits, int rows, int V, int64_t ldl, int k,
                             int32_t* argmax, int32_t* ids, float* vals, cudaStream_t st) {
    if (rows == 0) return cudaSuccess;
    int chunks = (V + kTopkChunk - 1) / kTopkChunk;
    // gridDim.y limit is 65535 rows per launch
    for (int r0 = 0; r0 < rows; r0 += 65535) {
        int nr = rows - r0 < 65535 ? rows - r0 : 65535;
        dim3 grid(chunks, nr);
        node_topk_kernel<<<grid, kTopkThreads, 0, st>>>(
            logits + (size_t)r0 * ldl, V, ldl, k, chunks, c->topk_cand + (size_t)r0 * chunks * kMaxK,
            c->row_counters + r0, argmax + r0, ids + (size_t)r0 * k, vals ? vals + (size_t)r0 * k : nullptr);
        c->launches++;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace goose
