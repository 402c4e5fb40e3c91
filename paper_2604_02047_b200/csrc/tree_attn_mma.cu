// Tree attention, warp-level tensor-core kernel (mma.sync m16n8k16 bf16, fp32 accumulate).
//
// Split-KV flash-decode: CTA (split, head, sequence) streams its share of the keys in 64-key tiles
// (cp.async, double buffered, zero-filled past the last valid row), each warp owns 16 query rows,
// scores stay in registers, the tree part of the mask comes from per-row 128-bit ancestor sets built
// from parent[] (Sec. 4 Stage 1: a node attends to the prefix and to its root-to-node ancestors).
// Partials (unnormalised O, running max, running sum) go to the workspace; the last CTA to arrive
// for a head (arrival counter, no spinning) combines them and writes bf16 output.
//
// This is the kernel for small trees and the safety net; the tcgen05 kernel handles large B.
#include "goose_internal.cuh"

namespace goose {

constexpr int kKT = 64;                    // keys per tile
constexpr int kLd = kHeadDim + 8;          // padded smem row (elements): 272 bytes, conflict-free ldmatrix
constexpr int kTileBytes = kKT * kLd * 2;  // one K or V tile
constexpr int kMmaSmem = 4 * kTileBytes;   // 2 stages x (K,V)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    int sz = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Ancestor set of node i as a 128-bit mask (bit j = node j is on the root-to-i path, i included).
// Assumes parent[] was validated (parent[0] = -1, 0 <= parent[v] < v), so the walk ends in <= B steps.
__device__ __forceinline__ void ancestor_mask(const int32_t* __restrict__ par, int i, int B, uint32_t (&m)[4]) {
    m[0] = m[1] = m[2] = m[3] = 0;
    int v = i;
    for (int step = 0; step < B && v >= 0; ++step) {
        uint32_t bit = 1u << (v & 31);
        int w = v >> 5;
        m[0] |= (w == 0) ? bit : 0; m[1] |= (w == 1) ? bit : 0;
        m[2] |= (w == 2) ? bit : 0; m[3] |= (w == 3) ? bit : 0;
        v = par[v];
    }
}
__device__ __forceinline__ bool mask_bit(const uint32_t (&m)[4], int j) {
    uint32_t w = (j < 32) ? m[0] : (j < 64) ? m[1] : (j < 96) ? m[2] : m[3];
    return (w >> (j & 31)) & 1u;
}

__device__ __forceinline__ void load_tile_async(unsigned char* smem_stage, const __nv_bfloat16* kc,
                                                const __nv_bfloat16* vc, int64_t row0, int key0, int n_keys,
                                                int H, int h, int tid, int nthreads) {
    // 64 rows x 16 chunks of 16 bytes, for K then V
    for (int c = tid; c < 2 * kKT * 16; c += nthreads) {
        int which = c >= kKT * 16;
        int cc = which ? c - kKT * 16 : c;
        int r = cc >> 4, ch = cc & 15;
        int key = key0 + r;
        bool valid = key < n_keys;
        const __nv_bfloat16* base = which ? vc : kc;
        const __nv_bfloat16* src = base + ((size_t)(row0 + (valid ? key : 0)) * H + h) * kHeadDim + ch * 8;
        uint32_t dst = smem_u32(smem_stage + which * kTileBytes + r * (kLd * 2) + ch * 16);
        cp_async16(dst, src, valid);
    }
}

__global__ void __launch_bounds__(256)
tree_attn_mma_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ kc,
                     const __nv_bfloat16* __restrict__ vc, const int64_t* __restrict__ row_off,
                     const int32_t* __restrict__ ctx_len, const int32_t* __restrict__ parent,
                     const int32_t* __restrict__ n_nodes, int Bcap, int H, int Hkv, int64_t kv_rows, float scale_log2, int splits,
                     float* __restrict__ partials, int32_t* __restrict__ head_counters,
                     int32_t* __restrict__ status, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_last;

    const int split = blockIdx.x, h = blockIdx.y, s = blockIdx.z;
    const int tid = threadIdx.x, nthreads = blockDim.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t4 = lane & 3;
    // grouped-query attention: query head h reads key/value head h / (H / Hkv); every query head streams its
    // key/value head by itself here (the tcgen05 kernel shares the stream across the group)
    const int hk = h / (H / Hkv);
    pdl_wait();
    pdl_trigger();
    // B = nodes of THIS sequence's tree (n_nodes[s] <= Bcap, the stride of q / out / parent); nodes beyond it do not
    // exist: nothing of theirs is read, their output rows are not written, their cache rows are past the last key
    const int B = nodes_of(n_nodes, s, Bcap);
    if (B == 0) {                                          // the sequence has left the batch (every CTA of it agrees)
        if (tid == 0 && split == 0 && h == 0 && nodes_bad(n_nodes, s, Bcap)) atomicOr(&status[s], GOOSE_ST_BAD_NODES);
        return;
    }
    const int ctx = max(ctx_len[s], 0);                    // device data: a negative length is treated as 0
    const int64_t row0 = row_off[s];
    const int n_keys = ctx + B;
    const int n_tiles = (n_keys + kKT - 1) / kKT;
    const int t_begin = (int)((long long)n_tiles * split / splits);
    const int t_end = (int)((long long)n_tiles * (split + 1) / splits);
    const int32_t* par = parent + (size_t)s * Bcap;

    // ---- validate parent[] (every CTA of the sequence reaches the same verdict)
    int bad = 0;
    for (int i = tid; i < B; i += nthreads) {
        int p = par[i];
        bad |= (i == 0) ? (p != -1) : (p < 0 || p >= i);
    }
    // the sequence's rows must lie inside the cache: never form an address from unchecked device data
    const bool bad_rows = ctx_len[s] < 0 || row0 < 0 || row0 + ctx + B > kv_rows;
    bad = __syncthreads_or(bad | (bad_rows ? 1 : 0));

    const int rowA = warp * 16 + g, rowB = rowA + 8;       // this thread's two query rows
    const bool warp_active = (warp * 16 < B) && !bad;
    uint32_t qf[8][4];
    uint32_t ancA[4], ancB[4];
    float o[16][4];
    float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
#pragma unroll
    for (int n = 0; n < 16; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }

    if (warp_active) {
        const uint32_t* qA = reinterpret_cast<const uint32_t*>(q + (((size_t)s * Bcap + (rowA < B ? rowA : 0)) * H + h) * kHeadDim);
        const uint32_t* qB = reinterpret_cast<const uint32_t*>(q + (((size_t)s * Bcap + (rowB < B ? rowB : 0)) * H + h) * kHeadDim);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qf[ks][0] = rowA < B ? qA[ks * 8 + t4] : 0u;
            qf[ks][1] = rowB < B ? qB[ks * 8 + t4] : 0u;
            qf[ks][2] = rowA < B ? qA[ks * 8 + 4 + t4] : 0u;
            qf[ks][3] = rowB < B ? qB[ks * 8 + 4 + t4] : 0u;
        }
        ancestor_mask(par, rowA < B ? rowA : 0, B, ancA);
        ancestor_mask(par, rowB < B ? rowB : 0, B, ancB);
    }

    // ---- stream the tiles
    if (t_begin < t_end && !bad) {
        load_tile_async(smem, kc, vc, row0, t_begin * kKT, n_keys, Hkv, hk, tid, nthreads);
    }
    cp_async_commit();
    for (int t = t_begin; t < t_end && !bad; ++t) {
        const int stage = (t - t_begin) & 1;
        if (t + 1 < t_end)
            load_tile_async(smem + (stage ^ 1) * 2 * kTileBytes, kc, vc, row0, (t + 1) * kKT, n_keys, Hkv, hk, tid, nthreads);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();

        if (warp_active) {
            const uint32_t k_base = smem_u32(smem + stage * 2 * kTileBytes);
            const uint32_t v_base = k_base + kTileBytes;
            float sc[8][4];
#pragma unroll
            for (int n = 0; n < 8; ++n) { sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f; }
            // S = Q K^T
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
                for (int np = 0; np < 4; ++np) {           // pairs of 8-key n-tiles
                    int mi = lane >> 3, r = lane & 7;
                    int key = 8 * (2 * np + (mi >> 1)) + r;
                    int d = 16 * ks + 8 * (mi & 1);
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4(b0, b1, b2, b3, k_base + key * (kLd * 2) + d * 2);
                    mma_bf16(sc[2 * np], qf[ks], b0, b1);
                    mma_bf16(sc[2 * np + 1], qf[ks], b2, b3);
                }
            }
            // scale, mask, online softmax (base-2 domain)
            const int key0 = t * kKT;
            const bool need_mask = key0 + kKT > ctx;
            float rmA = -INFINITY, rmB = -INFINITY;
#pragma unroll
            for (int n = 0; n < 8; ++n) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = sc[n][e] * scale_log2;
                    if (need_mask) {
                        int kk = key0 + 8 * n + 2 * t4 + (e & 1);
                        bool vis = kk < ctx;
                        if (!vis && kk < n_keys) vis = (e < 2) ? mask_bit(ancA, kk - ctx) : mask_bit(ancB, kk - ctx);
                        v = vis ? v : -INFINITY;
                    }
                    sc[n][e] = v;
                    if (e < 2) rmA = fmaxf(rmA, v); else rmB = fmaxf(rmB, v);
                }
            }
            rmA = fmaxf(rmA, __shfl_xor_sync(0xFFFFFFFFu, rmA, 1)); rmA = fmaxf(rmA, __shfl_xor_sync(0xFFFFFFFFu, rmA, 2));
            rmB = fmaxf(rmB, __shfl_xor_sync(0xFFFFFFFFu, rmB, 1)); rmB = fmaxf(rmB, __shfl_xor_sync(0xFFFFFFFFu, rmB, 2));
            float mnA = fmaxf(mA, rmA), mnB = fmaxf(mB, rmB);
            float muA = (mnA == -INFINITY) ? 0.f : mnA, muB = (mnB == -INFINITY) ? 0.f : mnB;
            float alA = exp2f(mA - muA), alB = exp2f(mB - muB);   // m = -inf -> 0
            mA = mnA; mB = mnB;
            lA *= alA; lB *= alB;
#pragma unroll
            for (int n = 0; n < 16; ++n) { o[n][0] *= alA; o[n][1] *= alA; o[n][2] *= alB; o[n][3] *= alB; }
            uint32_t pf[4][4];
#pragma unroll
            for (int n = 0; n < 8; ++n) {
                float p0 = exp2f(sc[n][0] - muA), p1 = exp2f(sc[n][1] - muA);
                float p2 = exp2f(sc[n][2] - muB), p3 = exp2f(sc[n][3] - muB);
                lA += p0 + p1; lB += p2 + p3;
                pf[n >> 1][(n & 1) * 2 + 0] = pack_bf16(p0, p1);
                pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
            }
            // O += P V
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {               // 16 keys per step
#pragma unroll
                for (int dp = 0; dp < 8; ++dp) {           // pairs of 8-wide d tiles
                    int key = 16 * kk + (lane & 7) + ((lane >> 3) & 1) * 8;
                    int d = 16 * dp + (lane >> 4) * 8;
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(b0, b1, b2, b3, v_base + key * (kLd * 2) + d * 2);
                    mma_bf16(o[2 * dp], pf[kk], b0, b1);
                    mma_bf16(o[2 * dp + 1], pf[kk], b2, b3);
                }
            }
        }
        __syncthreads();
    }
    cp_async_wait<0>();

    // ---- epilogue
    lA += __shfl_xor_sync(0xFFFFFFFFu, lA, 1); lA += __shfl_xor_sync(0xFFFFFFFFu, lA, 2);
    lB += __shfl_xor_sync(0xFFFFFFFFu, lB, 1); lB += __shfl_xor_sync(0xFFFFFFFFu, lB, 2);

    if (splits == 1 || bad) {
        if (bad) {
            if (tid == 0 && split == 0 && h == 0) atomicOr(&status[s], bad_rows ? GOOSE_ST_BAD_ROWS : GOOSE_ST_BAD_PARENT);
            // zero-fill this CTA's share of the head's output
            for (int idx = tid + split * nthreads; idx < B * (kHeadDim / 2); idx += nthreads * splits) {
                int i = idx / (kHeadDim / 2), c = idx % (kHeadDim / 2);
                reinterpret_cast<uint32_t*>(out + (((size_t)s * Bcap + i) * H + h) * kHeadDim)[c] = 0u;
                if (lse && c == 0) lse[((size_t)s * Bcap + i) * H + h] = 0.f;
            }
            return;
        }
        if (warp_active) {
            float iA = 1.f / lA, iB = 1.f / lB;
#pragma unroll
            for (int n = 0; n < 16; ++n) {
                if (rowA < B)
                    *reinterpret_cast<uint32_t*>(out + (((size_t)s * Bcap + rowA) * H + h) * kHeadDim + 8 * n + 2 * t4) = pack_bf16(o[n][0] * iA, o[n][1] * iA);
                if (rowB < B)
                    *reinterpret_cast<uint32_t*>(out + (((size_t)s * Bcap + rowB) * H + h) * kHeadDim + 8 * n + 2 * t4) = pack_bf16(o[n][2] * iB, o[n][3] * iB);
            }
            if (lse && t4 == 0) {
                if (rowA < B) lse[((size_t)s * Bcap + rowA) * H + h] = (mA + log2f(lA)) * kLn2;
                if (rowB < B) lse[((size_t)s * Bcap + rowB) * H + h] = (mB + log2f(lB)) * kLn2;
            }
        }
        return;
    }

    // split > 1: write the partial, then the last arriver combines
    const size_t head = (size_t)s * H + h;
    float* part = partials + (head * splits + split) * (size_t)kPartialFloats;
    if (warp * 16 < B) {
#pragma unroll
        for (int n = 0; n < 16; ++n) {
            if (rowA < B) *reinterpret_cast<float2*>(part + rowA * kHeadDim + 8 * n + 2 * t4) = make_float2(o[n][0], o[n][1]);
            if (rowB < B) *reinterpret_cast<float2*>(part + rowB * kHeadDim + 8 * n + 2 * t4) = make_float2(o[n][2], o[n][3]);
        }
        if (t4 == 0) {
            if (rowA < B) { part[kMaxB * kHeadDim + rowA] = mA; part[kMaxB * kHeadDim + kMaxB + rowA] = lA; }
            if (rowB < B) { part[kMaxB * kHeadDim + rowB] = mB; part[kMaxB * kHeadDim + kMaxB + rowB] = lB; }
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        int old = atomicAdd(&head_counters[head], 1);
        s_last = (old == splits - 1);
        if (s_last) head_counters[head] = 0;               // ready for the next launch
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const float* hp = partials + head * splits * (size_t)kPartialFloats;
    for (int idx = tid; idx < B * (kHeadDim / 2); idx += nthreads) {
        int i = idx / (kHeadDim / 2), c = idx % (kHeadDim / 2);
        float M = -INFINITY;
        for (int p = 0; p < splits; ++p) M = fmaxf(M, __ldcg(hp + p * (size_t)kPartialFloats + kMaxB * kHeadDim + i));
        float L = 0.f, a0 = 0.f, a1 = 0.f;
        for (int p = 0; p < splits; ++p) {
            const float* pp = hp + p * (size_t)kPartialFloats;
            float mp = __ldcg(pp + kMaxB * kHeadDim + i);
            float w = (mp == -INFINITY) ? 0.f : exp2f(mp - M);
            L += w * __ldcg(pp + kMaxB * kHeadDim + kMaxB + i);
            float2 ov = __ldcg(reinterpret_cast<const float2*>(pp + i * kHeadDim + 2 * c));
            a0 += w * ov.x; a1 += w * ov.y;
        }
        float inv = 1.f / L;
        reinterpret_cast<uint32_t*>(out + (((size_t)s * Bcap + i) * H + h) * kHeadDim)[c] = pack_bf16(a0 * inv, a1 * inv);
        if (lse && c == 0) lse[((size_t)s * Bcap + i) * H + h] = (M + log2f(L)) * kLn2;
    }
}

cudaError_t init_mma_kernel() {
    return cudaFuncSetAttribute(tree_attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMmaSmem);
}

int mma_splits(const goose_ctx* c, int S, int H) {
    // about two CTAs per SM in flight, at most 16 splits, and never more slots than the workspace holds
    int heads = S * H;
    int sp = (2 * c->num_sms + heads - 1) / heads;
    if (sp < 1) sp = 1;
    if (sp > 16) sp = 16;
    while (sp > 1 && (long long)heads * sp > c->n_slots) --sp;
    return sp;
}

cudaError_t launch_tree_attn_mma(goose_ctx* c, const __nv_bfloat16* q, const __nv_bfloat16* kc,
                                 const __nv_bfloat16* vc, int64_t kv_rows, const int64_t* row_off, const int32_t* ctx_len,
                                 const int32_t* parent, const int32_t* n_nodes, int S, int B, int H, int Hkv, float scale,
                                 __nv_bfloat16* out, float* lse, cudaStream_t st) {
    if (S == 0 || H == 0) return cudaSuccess;
    int splits = mma_splits(c, S, H);
    int warps = (B + 15) / 16;
    if (warps < 4) warps = 4;
    dim3 grid(splits, H, S);
    cudaError_t e = launch_pdl(tree_attn_mma_kernel, grid, dim3(warps * 32), kMmaSmem, st, q, kc, vc, row_off, ctx_len,
                               parent, n_nodes, B, H, Hkv, kv_rows, scale * kLog2e, splits, c->partials, c->head_counters, c->status, out, lse);
    c->launches++;
    return e;
}

}  // namespace goose
