// Pieces of the tensor-core attention path that two kernels share: the work partition of the persistent main kernel
// and the merge of its split-KV partials.  The merge runs either as a kernel of its own (goose_tree_attn) or as a block
// role of the step's last launch (goose_verify_step), where it overlaps the acceptance walk and the compaction instead
// of standing between the attention kernel and the top-k.
#pragma once

#include <cuda_fp16.h>

#include "goose_internal.cuh"

namespace goose {

constexpr int kTile = 128;                       // keys per tile
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kCombineThreads = 256;
constexpr int kCombineRound = 4;                 // partials merged per load round of the merge
// split-KV partial of the main kernel: normalised O/l as fp16, uint4 [16 column groups of 8][128 rows] (32 KB, a warp's
// stores and the merge's loads are contiguous), then m[128], l[128] as fp32
constexpr int kPartHalfWords = 16 * 128 * 4;     // 32-bit words of the fp16 block
constexpr int kUmmaPartFloats = kPartHalfWords + 2 * kMaxB;

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// ---------------------------------------------------------------- work partition (same code in every role)
struct Work {
    const int32_t* ctx_len;
    const int32_t* n_nodes;   // per-sequence node counts, or NULL (every tree has B nodes)
    int S, H, B, G;           // H = heads of the work list = M tiles x key/value heads (M-tile-major)
    long long total;          // all items
    bool small;               // total * (G + 1) fits 31 bits: 32-bit arithmetic (64-bit division is slow on the GPU)
    // ctx_len comes from device memory: a negative value is treated as 0 (the tree rows alone).  A sequence's keys are
    // its prefix and the nodes its tree really has; a sequence without nodes (it has left the batch) has no items.
    __device__ __forceinline__ int tiles(int s) const {
        if (!n_nodes) return (max(ctx_len[s], 0) + B + kTile - 1) / kTile;
        const int nn = nodes_of(n_nodes, s, B);
        return nn == 0 ? 0 : (max(ctx_len[s], 0) + nn + kTile - 1) / kTile;
    }
    __device__ __forceinline__ void init() {
        long long tot = 0;
        for (int s = 0; s < S; ++s) tot += (long long)H * tiles(s);
        total = tot;
        small = tot * (G + 1) < 0x7FFFFFFFll;
    }
    __device__ __forceinline__ long long cta_start(int c) const {
        if (small) return ((uint32_t)total * (uint32_t)c) / (uint32_t)G;
        return total * c / G;
    }
    __device__ __forceinline__ int cta_of(long long w) const {
        int c = small ? (int)(((uint32_t)w * (uint32_t)G) / (uint32_t)total) : (int)(w * G / total);
        if (c >= G) c = G - 1;
        while (c + 1 < G && cta_start(c + 1) <= w) ++c;
        while (c > 0 && cta_start(c) > w) --c;
        return c;
    }
};

struct Cursor {               // walks items in order
    long long w;              // item index
    int s, h, t, T;
    __device__ __forceinline__ void seek(const Work& wk, long long w0) {
        long long off = 0;
        int ss = 0;
        int TT = wk.tiles(0);
        while (ss + 1 < wk.S && off + (long long)wk.H * TT <= w0) {
            off += (long long)wk.H * TT;
            ++ss;
            TT = wk.tiles(ss);
        }
        s = ss; T = TT; w = w0;
        const long long rem = w0 - off;
        h = wk.small ? (int)((uint32_t)rem / (uint32_t)TT) : (int)(rem / TT);
        t = (int)(rem - (long long)h * TT);
    }
    __device__ __forceinline__ void next(const Work& wk) {
        ++w; ++t;
        if (t == T) {
            t = 0; ++h;
            if (h == wk.H) {                              // next sequence that has any items
                h = 0; ++s;
                if (!wk.n_nodes) { if (s < wk.S) T = wk.tiles(s); }
                else while (s < wk.S && (T = wk.tiles(s)) == 0) ++s;
            }
        }
    }
};

// ---------------------------------------------------------------- merge of the split-KV partials
// One call handles 32 rows (rg = row group) of head h (a head of the work list = M tile x key/value head) of sequence s
// with 256 threads.  A head that one CTA of the main kernel covered entirely was written directly and is skipped; any
// other is the merge of its CTAs' partials:
//   M = max m_p,  L = sum l_p 2^(m_p - M),  out = sum_p 2^(m_p - M) O_p / L.
// Lane <-> row (coalesced float4 loads of the transposed partial layout), warp <-> 16 output columns.
// The function contains the caller's dependency wait (pdl_wait / pdl_trigger): everything in front of it needs only
// ctx_len[] and n_nodes[].
struct CombineArgs {
    const int32_t* ctx_len;
    const int32_t* n_nodes;
    int S, B, H, Hkv, g, nb;
    int G;                    // CTAs of the main kernel
    int Hw;                   // heads of the work list
    const float* partials;
    __nv_bfloat16* out;
    float* lse;
};

template <bool kGrouped, bool kCounts>
__device__ __forceinline__ void combine_heads(const CombineArgs& ca, int rg, int h, int s) {
    const int32_t* __restrict__ ctx_len = ca.ctx_len;
    const int32_t* __restrict__ n_nodes = kCounts ? ca.n_nodes : nullptr;
    const int S = ca.S, B = ca.B, H = ca.H, G = ca.G;
    const float* __restrict__ partials = ca.partials;
    __nv_bfloat16* __restrict__ out = ca.out;
    float* __restrict__ lse = ca.lse;
    const int Hkv_arg = ca.Hkv, g_arg = ca.g, nb_arg = ca.nb;

    const int Hkv = kGrouped ? Hkv_arg : H, g = kGrouped ? g_arg : 1, nb = kGrouped ? nb_arg : B;
    const int Hw = ca.Hw;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // The partition arithmetic needs only ctx_len[], which is final before this kernel's CTAs can start: the main
    // kernel triggers its dependents after its own pdl_wait(), i.e. after whatever produced ctx_len[] completed.
    // So all of it runs before the wait, and the partial loads are issued the moment the main grid is done.
    Work wk;
    wk.ctx_len = ctx_len; wk.n_nodes = n_nodes; wk.S = S; wk.H = Hw; wk.B = B; wk.G = G;
    wk.init();
    long long off = 0;
    for (int ss = 0; ss < s; ++ss) off += (long long)Hw * wk.tiles(ss);
    const int T = wk.tiles(s);                             // 0: the sequence has no nodes, hence no items and no output
    const long long head_first = off + (long long)h * T;
    const bool any = !kCounts || T > 0;                    // (without counts every sequence has tiles)
    const int c_lo = any ? wk.cta_of(head_first) : 0, c_hi = any ? wk.cta_of(head_first + T - 1) : 0;
    const bool whole = c_lo == c_hi;                       // written directly by the main kernel (or nothing to write)
    const int row = rg * 32 + lane;                        // row of the M tile = (node of the tile, head of the group)
    const int mt = kGrouped ? h / Hkv : 0, hk = h - mt * Hkv;
    const int i_local = kGrouped ? row / g : row, node = mt * nb + i_local;
    const int hq = hk * g + (row - i_local * g);
    const bool row_valid = i_local < nb && node < nodes_of(n_nodes, s, B);
    // CTA c's partial for this head sits in slot 2c, or 2c+1 when its segment starts at the head's first tile,
    // which only the first CTA can do.  With fewer items than CTAs some CTAs in [c_lo, c_hi] are empty.
    const int flag_lo = wk.cta_start(c_lo) <= head_first ? 1 : 0;
    const bool sparse = wk.total < G;
    // every CTA waits, also those with nothing to do: the next kernel in the stream relies on "this grid is
    // complete" implying "the main grid is complete"
    pdl_wait();                                            // the main kernel's partials are complete and visible
    pdl_trigger();
    if (whole || !row_valid) return;
    float M_run = -INFINITY, L_run = 0.f;
    float acc[16];                                         // warp w owns columns 16w .. 16w+15 (column groups 2w, 2w+1)
#pragma unroll
    for (int u = 0; u < 16; ++u) acc[u] = 0.f;

    // kCombineRound parts per round: their (m, l) and their two 16-byte pieces of O/l are loaded together
    // (16 independent loads in flight per thread); a running (M, L) with rescaling merges the rounds
    for (int cb = c_lo; cb <= c_hi; cb += kCombineRound) {
        float mp[kCombineRound], lp[kCombineRound];
        uint4 x[kCombineRound][2];
#pragma unroll
        for (int q = 0; q < kCombineRound; ++q) {
            const int c = cb + q;
            bool use = c <= c_hi;
            if (use && sparse) use = wk.cta_start(c + 1) > wk.cta_start(c);
            const int sl = use ? 2 * c + (c == c_lo ? flag_lo : 0) : 0;
            const float* pp = partials + (size_t)sl * kUmmaPartFloats;
            mp[q] = use ? __ldcg(pp + kPartHalfWords + row) : -INFINITY;
            lp[q] = use ? __ldcg(pp + kPartHalfWords + kMaxB + row) : 0.f;
            const uint4* p4 = reinterpret_cast<const uint4*>(pp) + row;
#pragma unroll
            for (int u = 0; u < 2; ++u)
                x[q][u] = use ? __ldcg(p4 + (2 * warp + u) * 128) : make_uint4(0u, 0u, 0u, 0u);
        }
        float M_new = M_run;
#pragma unroll
        for (int q = 0; q < kCombineRound; ++q) M_new = fmaxf(M_new, mp[q]);
        const float a_old = (M_run == -INFINITY) ? 0.f : ex2(M_run - M_new);
        L_run *= a_old;
#pragma unroll
        for (int u = 0; u < 16; ++u) acc[u] *= a_old;
#pragma unroll
        for (int q = 0; q < kCombineRound; ++q) {
            const float w = ((mp[q] == -INFINITY) ? 0.f : ex2(mp[q] - M_new)) * lp[q];   // un-normalise: O_p = x_p * l_p
            L_run += w;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const uint32_t hw[4] = {x[q][u].x, x[q][u].y, x[q][u].z, x[q][u].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&hw[e]));
                    acc[8 * u + 2 * e] += w * f.x;
                    acc[8 * u + 2 * e + 1] += w * f.y;
                }
            }
        }
        M_run = M_new;
    }
    const float inv = 1.f / L_run;
    uint4* dst = reinterpret_cast<uint4*>(out + (((size_t)s * B + node) * H + hq) * kHeadDim + 16 * warp);
#pragma unroll
    for (int u = 0; u < 2; ++u)
        dst[u] = make_uint4(pack_bf16x2(acc[8 * u] * inv, acc[8 * u + 1] * inv), pack_bf16x2(acc[8 * u + 2] * inv, acc[8 * u + 3] * inv),
                            pack_bf16x2(acc[8 * u + 4] * inv, acc[8 * u + 5] * inv), pack_bf16x2(acc[8 * u + 6] * inv, acc[8 * u + 7] * inv));
    if (lse && warp == 0) lse[((size_t)s * B + node) * H + hq] = (M_run + log2f(L_run)) * kLn2;
}

// the merge as a kernel of its own: grid (row groups of 32, heads of the work list, S)
template <bool kGrouped, bool kCounts>
__global__ void __launch_bounds__(kCombineThreads)
tree_attn_combine_kernel(const CombineArgs ca) {
    combine_heads<kGrouped, kCounts>(ca, blockIdx.x, blockIdx.y, blockIdx.z);
}

// host side: what the merge needs to know about the main kernel's launch (filled by launch_tree_attn_umma)
struct CombinePlan {
    CombineArgs args;
    int row_groups;           // blocks per head
    bool grouped;
    bool valid;               // false: nothing to merge (no tensor-core launch happened)
};

}  // namespace goose
