// Tree attention on the 5th-generation tensor cores: persistent, warp-specialised kernel
// (tcgen05.mma with TMEM accumulators, TMA loads, mbarrier pipeline).
//
// Work = all (sequence, head, 128-key tile) items in sequence-major order, dealt to the CTAs
// (one per SM) in contiguous ranges, so every SM streams the same number of K/V bytes.  A run of
// items of one head inside a CTA's range is a "segment"; a segment that covers its whole head
// writes the bf16 output directly, any other segment writes a partial (O / l as fp16, running max m and
// running sum l as fp32) to the workspace, and a small second kernel (tree_attn_combine_kernel, spread
// over all SMs) merges the partials of every head that was split.
//
// Roles (192 threads):
//   warp 0, lane 0   TMA producer: Q of the segment, then K and V tiles into a ring of 32 KB stages
//   warp 1, lane 0   MMA issuer:   S = Q K^T into TMEM (double buffered), O += P V into TMEM with P read
//                                  from tensor memory
//   warps 2..5       softmax:      one query row per thread (TMEM lane = row): S from TMEM, ancestor
//                                  mask on the tiles that reach the tree rows, exp2, P (bf16) written back
//                                  over the first 64 columns of the S buffer it came from, lazy rescaling
//                                  of O in TMEM, epilogue (output or partial).
// All B <= 128 query rows ride in one M = 128 MMA; rows >= B compute on don't-care data and are
// never written out.  Grouped-query attention (H query heads over Hkv key/value heads, g = H / Hkv) stacks the g
// query heads of a group into the same M tile -- row r = (node r / g, group member r % g) -- so a K/V tile is
// streamed once per group; when B * g > 128 the nodes are cut into M tiles of floor(128 / g) nodes and the K/V of a
// head is streamed once per M tile.  A "head" of the work list below is one (M tile, key/value head) pair.
// The tree part of the mask (Sec. 4 Stage 1: a node attends to the prefix and to its root-to-node ancestors) is a
// per-row 128-bit ancestor set built from parent[].
//
// Every wait in this file is bounded: when a wait runs out of polls the CTA raises an abort flag,
// sets GOOSE_ST_TIMEOUT, drains its own copies in flight (again bounded), frees its TMEM and returns.
#include <cuda.h>
#include <cuda_fp16.h>

#include "goose_internal.cuh"
#include "tree_attn_combine.cuh"

namespace goose {

namespace {

constexpr int kStages = 5;                      // ring of K/V stages (P lives in tensor memory, not here)
constexpr int kStageBytes = kTile * kHeadDim * 2;   // 32 KB: one K or one V tile
constexpr int kHalfBytes = kTile * 128;         // 16 KB: 128 rows x 64 bf16 (one swizzle-atom column)
constexpr int kQBytes = 2 * kHalfBytes;
constexpr int kHeaderBytes = 1024;
constexpr int kUmmaSmem = kHeaderBytes + 1024 /*alignment slack*/ + 2 * kQBytes + kStages * kStageBytes;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColO = 256;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;       // rescale O only when the running max grew by > 2^8
constexpr long long kWaitCycles = 2000000000ll;  // bound of every wait: about one second of SM clock

struct Header {                                  // lives at the start of dynamic shared memory
    unsigned long long kv_full[kStages];
    unsigned long long kv_empty[kStages];
    unsigned long long q_full[2], q_empty[2];    // Q is double buffered: the next segment's Q is prefetched
    unsigned long long s_full[2];
    unsigned long long p_ready, pv_done, o_free;
    unsigned long long group_bar;                // barrier of the 128 softmax threads (bounded, unlike bar.sync)
    uint32_t tmem_base;
    volatile int abort_flag;
    int bad_parent;
    int par[kMaxB];                              // parent[] of the current segment's sequence
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false, and raises the CTA's abort flag, when `limit` SM cycles pass without the barrier
// completing; returns false at once when another role has already aborted.
__device__ __forceinline__ bool mbar_wait_limit(Header* hd, unsigned long long* bar, uint32_t parity, int32_t* status,
                                                long long limit) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (hd->abort_flag) return false;
        if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > limit) break;
    }
    hd->abort_flag = 1;
    atomicOr(status, GOOSE_ST_TIMEOUT);
    return false;
}
// every wait of the attention kernel: about one second of SM clock
__device__ __forceinline__ bool mbar_wait(Header* hd, unsigned long long* bar, uint32_t parity, int32_t* status) {
    return mbar_wait_limit(hd, bar, parity, status, kWaitCycles);
}
// Bounded wait used only while draining after an abort (ignores the abort flag).
__device__ __forceinline__ void mbar_drain(unsigned long long* bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity) && clock64() - t0 < kWaitCycles) {}
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, unsigned long long* bar,
                                            int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_3d_hint(void* dst, const CUtensorMap* map, unsigned long long* bar,
                                                 int c0, int c1, int c2, unsigned long long policy) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
                 "[%0], [%1, {%3, %4, %5}], [%2], %6;"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
__device__ __forceinline__ unsigned long long l2_policy_evict_first() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// shared-memory matrix descriptor, 128-byte swizzle; addresses and offsets in bytes
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr >> 4) & 0x3FFF) | ((uint64_t)((lbo >> 4) & 0x3FFF) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3FFF) << 32) | (1ull << 46) /*descriptor version*/ | (2ull << 61) /*SWIZZLE_128B*/;
}
// instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128, A K-major, B K-major or MN-major
__host__ __device__ constexpr uint32_t instr_desc(bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// same, with the A operand (M x 16 bf16, two per 32-bit column, lane = row) read from tensor memory
__device__ __forceinline__ void umma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

#define TMEM_LD32(taddr, v, off)                                                                                      \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                            \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                          \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                           \
                 : "=r"(v[off + 0]), "=r"(v[off + 1]), "=r"(v[off + 2]), "=r"(v[off + 3]), "=r"(v[off + 4]),          \
                   "=r"(v[off + 5]), "=r"(v[off + 6]), "=r"(v[off + 7]), "=r"(v[off + 8]), "=r"(v[off + 9]),          \
                   "=r"(v[off + 10]), "=r"(v[off + 11]), "=r"(v[off + 12]), "=r"(v[off + 13]), "=r"(v[off + 14]),     \
                   "=r"(v[off + 15]), "=r"(v[off + 16]), "=r"(v[off + 17]), "=r"(v[off + 18]), "=r"(v[off + 19]),     \
                   "=r"(v[off + 20]), "=r"(v[off + 21]), "=r"(v[off + 22]), "=r"(v[off + 23]), "=r"(v[off + 24]),     \
                   "=r"(v[off + 25]), "=r"(v[off + 26]), "=r"(v[off + 27]), "=r"(v[off + 28]), "=r"(v[off + 29]),     \
                   "=r"(v[off + 30]), "=r"(v[off + 31])                                                               \
                 : "r"(taddr))
#define TMEM_ST32(taddr, v, off)                                                                                      \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "                                                     \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                          \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"                                  \
                 ::"r"(v[off + 0]), "r"(v[off + 1]), "r"(v[off + 2]), "r"(v[off + 3]), "r"(v[off + 4]),               \
                   "r"(v[off + 5]), "r"(v[off + 6]), "r"(v[off + 7]), "r"(v[off + 8]), "r"(v[off + 9]),               \
                   "r"(v[off + 10]), "r"(v[off + 11]), "r"(v[off + 12]), "r"(v[off + 13]), "r"(v[off + 14]),          \
                   "r"(v[off + 15]), "r"(v[off + 16]), "r"(v[off + 17]), "r"(v[off + 18]), "r"(v[off + 19]),          \
                   "r"(v[off + 20]), "r"(v[off + 21]), "r"(v[off + 22]), "r"(v[off + 23]), "r"(v[off + 24]),          \
                   "r"(v[off + 25]), "r"(v[off + 26]), "r"(v[off + 27]), "r"(v[off + 28]), "r"(v[off + 29]),          \
                   "r"(v[off + 30]), "r"(v[off + 31]), "r"(taddr) : "memory")

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// barrier of the 128 softmax threads; `n` counts its uses (every thread calls it the same number of times)
__device__ __forceinline__ bool group_sync(Header* hd, uint32_t& n, int32_t* status) {
    mbar_arrive(&hd->group_bar);
    bool ok = mbar_wait(hd, &hd->group_bar, n & 1, status);
    ++n;
    return ok;
}

// ---------------------------------------------------------------- the kernel
// kGrouped = false is multi-head attention: one query head per key/value head and one M tile per sequence are
// compile-time facts there (the per-row index arithmetic folds away); kGrouped = true takes them from the arguments.
// kCounts = false is the instantiation for n_nodes == NULL: the counts fold away at compile time
template <bool kGrouped, bool kCounts>
__global__ void __launch_bounds__(kThreads, 1)
tree_attn_umma_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                      const __grid_constant__ CUtensorMap tmap_v, const int64_t* __restrict__ row_off,
                      const int32_t* __restrict__ ctx_len, const int32_t* __restrict__ parent,
                      const int32_t* __restrict__ n_nodes,
                      int S, int B, int H, int Hkv_arg, int g_arg, int nb_arg, int64_t kv_rows, float scale_log2,
                      float* __restrict__ partials,
                      int32_t* __restrict__ status,
                      __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    if (!kCounts) n_nodes = nullptr;

    const int Hkv = kGrouped ? Hkv_arg : H, g = kGrouped ? g_arg : 1, nb = kGrouped ? nb_arg : B;
    extern __shared__ unsigned char smem_raw[];
    Header* hd = reinterpret_cast<Header*>(smem_raw);
    unsigned char* buf = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + kHeaderBytes + 1023) & ~(uintptr_t)1023);
    unsigned char* q_smem = buf;
    unsigned char* kv_smem = buf + 2 * kQBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- set-up
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&hd->kv_full[i], 1); mbar_init(&hd->kv_empty[i], 1); }
        mbar_init(&hd->q_full[0], 1); mbar_init(&hd->q_full[1], 1);
        mbar_init(&hd->q_empty[0], 1); mbar_init(&hd->q_empty[1], 1);
        mbar_init(&hd->s_full[0], 1); mbar_init(&hd->s_full[1], 1);
        mbar_init(&hd->p_ready, 128); mbar_init(&hd->pv_done, 1); mbar_init(&hd->o_free, 128);
        mbar_init(&hd->group_bar, 128);
        hd->abort_flag = 0; hd->bad_parent = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {                                   // TMEM: the whole 512 columns (one CTA per SM)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&hd->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = hd->tmem_base;
    // L2 prefetch hints for the small index arrays (a hint reads no data, so it may precede the wait)
    if (threadIdx.x == 32) {
        asm volatile("prefetch.global.L2 [%0];" ::"l"(ctx_len));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(row_off));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(parent));
    }
    // everything above touched no global memory: now wait for the preceding kernel, then let the next
    // one (the combine kernel) get resident early -- it waits for this grid before reading the partials
    pdl_wait();
    pdl_trigger();
    if (n_nodes && blockIdx.x == 0 && threadIdx.x == 33)   // an idle lane reports node counts outside [0, B] (read as 0)
        for (int s = 0; s < S; ++s)
            if (nodes_bad(n_nodes, s, B)) atomicOr(&status[s], GOOSE_ST_BAD_NODES);
    Work wk;
    // g query heads per key/value head, nb nodes per M tile (nb * g <= 128), n_mt M tiles per sequence
    const int n_mt = kGrouped ? (B + nb - 1) / nb : 1;
    wk.ctx_len = ctx_len; wk.n_nodes = n_nodes; wk.S = S; wk.H = n_mt * Hkv; wk.B = B; wk.G = gridDim.x;
    wk.init();
    const long long w_begin = wk.cta_start(blockIdx.x), w_end = wk.cta_start(blockIdx.x + 1);


    if (w_begin < w_end) {
        if (warp == 0) {
            // =========================================================== TMA producer
            if (lane == 0) {
                prefetch_tmap(&tmap_q); prefetch_tmap(&tmap_k); prefetch_tmap(&tmap_v);
                // K and V are read exactly once: mark them evict-first so that the split-KV partials
                // (written and re-read within this launch) stay resident in L2
                const unsigned long long pol_stream = l2_policy_evict_first();
                Cursor cu; cu.seek(wk, w_begin);
                uint32_t ring = 0, seg = 0;
                bool ok = true;
                while (ok && cu.w < w_end) {
                    const int64_t row0 = row_off[cu.s];
                    // Q of this segment
                    const uint32_t qb = seg & 1;           // seg = index of this segment
                    ok = mbar_wait(hd, &hd->q_empty[qb], ((seg >> 1) & 1) ^ 1, status);
                    if (!ok) break;
                    // box = nb nodes x g heads x 64 dims: lands as rows r = node * g + member (rows past the
                    // sequence's last node hold the next sequence's queries or the zero fill: never written out)
                    const int mt = kGrouped ? cu.h / Hkv : 0, hk = cu.h - mt * Hkv;
                    mbar_expect_tx(&hd->q_full[qb], (uint32_t)(nb * g) * 256u);
                    tma_load_4d(q_smem + qb * kQBytes, &tmap_q, &hd->q_full[qb], 0, 0, hk, cu.s * B + mt * nb);
                    tma_load_4d(q_smem + qb * kQBytes + kHalfBytes, &tmap_q, &hd->q_full[qb], 64, 0, hk, cu.s * B + mt * nb);
                    ++seg;                                 // segments whose Q load has been issued
                    const int s0 = cu.s, h0 = cu.h;
                    while (ok && cu.w < w_end && cu.s == s0 && cu.h == h0) {
                        const int krow = (int)(row0 + (int64_t)cu.t * kTile);
                        for (int kv = 0; kv < 2 && ok; ++kv) {
                            const uint32_t st = ring % kStages, fill = ring / kStages;
                            ok = mbar_wait(hd, &hd->kv_empty[st], (fill & 1) ^ 1, status);
                            if (!ok) break;
                            unsigned char* dst = kv_smem + st * kStageBytes;
                            mbar_expect_tx(&hd->kv_full[st], kStageBytes);
                            const CUtensorMap* mp = kv ? &tmap_v : &tmap_k;
                            tma_load_3d_hint(dst, mp, &hd->kv_full[st], 0, hk, krow, pol_stream);
                            tma_load_3d_hint(dst + kHalfBytes, mp, &hd->kv_full[st], 64, hk, krow, pol_stream);
                            ++ring;
                        }
                        cu.next(wk);
                    }
                }
                if (!ok) {
                    // aborted: drain this thread's copies still in flight (bounded) before the CTA exits
                    uint32_t first = ring > kStages ? ring - kStages : 0;
                    for (uint32_t r = first; r < ring; ++r) mbar_drain(&hd->kv_full[r % kStages], (r / kStages) & 1);
                    if (seg > 0) mbar_drain(&hd->q_full[(seg - 1) & 1], ((seg - 1) >> 1) & 1);
                    if (seg > 1) mbar_drain(&hd->q_full[(seg - 2) & 1], ((seg - 2) >> 1) & 1);
                }
            }
        } else if (warp == 1) {
            // =========================================================== MMA issuer
            if (lane == 0) {
                Cursor cu; cu.seek(wk, w_begin);
                uint32_t jg = 0, seg = 0;                  // CTA-global tile and segment counters
                bool ok = true;
                const uint32_t q_base = smem_u32(q_smem), kv_addr = smem_u32(kv_smem);
                constexpr uint32_t idesc_qk = instr_desc(false), idesc_pv = instr_desc(true);

                auto issue_pv = [&](uint32_t j, bool first_of_segment) -> bool {
                    // tile j's P (bf16) has replaced S(j) in the first 64 columns of its S buffer
                    if (!mbar_wait(hd, &hd->p_ready, j & 1, status)) return false;
                    const uint32_t ring = 2 * j + 1, st = ring % kStages;
                    if (!mbar_wait(hd, &hd->kv_full[st], (ring / kStages) & 1, status)) return false;
                    if (first_of_segment && seg > 0)       // the previous segment's O must have left TMEM
                        if (!mbar_wait(hd, &hd->o_free, (seg - 1) & 1, status)) return false;
                    tc_fence_after();
                    const uint32_t v_addr = kv_addr + st * kStageBytes;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {       // 16 keys per instruction
                        uint64_t b = smem_desc(v_addr + kk * 2048, kHalfBytes, 1024);   // MN-major: LBO = next 64 d
                        umma_f16_ts(tmem + kColO, tmem + kColS + (j & 1) * 128 + kk * 8, b, idesc_pv,
                                    (!first_of_segment || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(&hd->kv_empty[st]);
                    umma_commit(&hd->pv_done);
                    return true;
                };

                while (ok && cu.w < w_end) {
                    ok = mbar_wait(hd, &hd->q_full[seg & 1], (seg >> 1) & 1, status);
                    if (!ok) break;
                    const uint32_t q_addr = q_base + (seg & 1) * kQBytes;
                    const int s0 = cu.s, h0 = cu.h;
                    const uint32_t j_first = jg;
                    while (ok && cu.w < w_end && cu.s == s0 && cu.h == h0) {
                        const uint32_t ring = 2 * jg, st = ring % kStages;
                        ok = mbar_wait(hd, &hd->kv_full[st], (ring / kStages) & 1, status);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t k_addr = kv_addr + st * kStageBytes;
                        const uint32_t d_tmem = tmem + kColS + (jg & 1) * 128;
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {   // 16 of the 128 head dims per instruction
                            uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                            umma_f16(d_tmem, smem_desc(q_addr + off, 16, 1024), smem_desc(k_addr + off, 16, 1024),
                                     idesc_qk, kk > 0 ? 1u : 0u);
                        }
                        umma_commit(&hd->s_full[jg & 1]);
                        umma_commit(&hd->kv_empty[st]);
                        if (jg > j_first) ok = issue_pv(jg - 1, jg - 1 == j_first);
                        ++jg;
                        cu.next(wk);
                    }
                    if (!ok) break;
                    umma_commit(&hd->q_empty[seg & 1]);    // every QK^T of the segment has been issued
                    ok = issue_pv(jg - 1, jg - 1 == j_first);
                    ++seg;
                }
            }
        } else {
            // =========================================================== softmax / epilogue (128 threads)
            const int row = 32 * (warp & 3) + lane;        // TMEM lane == query row
            const uint32_t lane_sel = (uint32_t)(32 * (warp & 3)) << 16;
            const int i_local = kGrouped ? row / g : row;  // row = (node of the M tile, head of the group)
            const int member = row - i_local * g;
            const int sm_tid = threadIdx.x - 64;           // 0..127
            Cursor cu; cu.seek(wk, w_begin);
            uint32_t jg = 0, seg = 0, gsync = 0;
            bool ok = true;
            uint32_t v[128];
            int cur_s = -1, cur_mt = -1;
            bool bad = false;
            uint32_t anc[4] = {0, 0, 0, 0};

            while (ok && cu.w < w_end) {
                const int s0 = cu.s, h0 = cu.h, T = cu.T;
                const int mt = kGrouped ? h0 / Hkv : 0, hk = h0 - mt * Hkv;
                const int node = mt * nb + i_local;        // tree node of this thread's row
                const int nn = nodes_of(n_nodes, s0, B);   // nodes this sequence's tree really has (> 0: it has items)
                const bool row_valid = i_local < nb && node < nn;
                const bool warp_has_rows = 32 * (warp & 3) < min(nb, nn - mt * nb) * g;
                const int ctx = max(ctx_len[s0], 0);
                const int n_keys = ctx + nn;               // rows behind may hold anything: masked, and zeroed in V
                const int32_t* par = parent + (size_t)s0 * B;
                const int t_first = cu.t;
                // new sequence: validate parent[] (all 128 threads reach the same verdict) and rebuild
                // this row's ancestor set; consecutive segments of one sequence reuse both
                const bool new_seq = s0 != cur_s;
                if (new_seq) {
                    cur_s = s0;
                    if (row < nn) {                        // thread r stages parent[r] (independent of the row stacking)
                        int p = par[row];
                        hd->par[row] = p;
                        if ((row == 0) ? (p != -1) : (p < 0 || p >= row)) hd->bad_parent = 1;
                    }
                    // the sequence's rows must lie inside the cache (TMA would only read zeros outside, but the
                    // result would be meaningless): treated like an invalid tree, with its own status bit
                    const int64_t r0 = row_off[s0];
                    const bool bad_rows = ctx_len[s0] < 0 || r0 < 0 || r0 + ctx + nn > kv_rows;
                    if (bad_rows && sm_tid == 0) { hd->bad_parent = 1; atomicOr(&status[s0], GOOSE_ST_BAD_ROWS); }
                    ok = group_sync(hd, gsync, status);
                    bad = hd->bad_parent != 0;
                    ok = ok && group_sync(hd, gsync, status);
                    if (!ok) break;
                    if (sm_tid == 0 && bad) { hd->bad_parent = 0; if (!bad_rows) atomicOr(&status[s0], GOOSE_ST_BAD_PARENT); }
                }
                if (new_seq || mt != cur_mt) {             // hd->par[] still holds this sequence's parents
                    cur_mt = mt;
                    anc[0] = anc[1] = anc[2] = anc[3] = 0;
                    if (row_valid) {
                        if (bad) {
                            const uint32_t bit = 1u << (node & 31);
                            const int wsel = node >> 5;
                            anc[0] = (wsel == 0) ? bit : 0; anc[1] = (wsel == 1) ? bit : 0;
                            anc[2] = (wsel == 2) ? bit : 0; anc[3] = (wsel == 3) ? bit : 0;
                        } else {
                            int vtx = node;
                            for (int step = 0; step < B && vtx >= 0; ++step) {
                                uint32_t bit = 1u << (vtx & 31);
                                int wsel = vtx >> 5;
                                anc[0] |= (wsel == 0) ? bit : 0; anc[1] |= (wsel == 1) ? bit : 0;
                                anc[2] |= (wsel == 2) ? bit : 0; anc[3] |= (wsel == 3) ? bit : 0;
                                vtx = hd->par[vtx];
                            }
                        }
                    }
                }
                float m_run = -INFINITY, l_run = 0.f;
                int seg_tiles = 0;

                while (ok && cu.w < w_end && cu.s == s0 && cu.h == h0) {
                    const int t = cu.t;
                    const bool first = (t == t_first);
                    ok = mbar_wait(hd, &hd->s_full[jg & 1], (jg >> 1) & 1, status);
                    if (!ok) break;
                    tc_fence_after();
                    float m_use = 0.f;
                    if (warp_has_rows) {
                        const uint32_t s_addr = tmem + kColS + (jg & 1) * 128 + lane_sel;
                        TMEM_LD32(s_addr, v, 0); TMEM_LD32(s_addr + 32, v, 32);
                        TMEM_LD32(s_addr + 64, v, 64); TMEM_LD32(s_addr + 96, v, 96);
                        tmem_wait_ld();
                        const int key0 = t * kTile;
                        if (key0 + kTile > ctx) {          // this tile reaches the tree rows (or the ragged end)
                            // visibility of the tile's 128 keys as one 128-bit mask: the prefix keys
                            // (c < ctx - key0) and the ancestor set shifted to where the tree rows start
                            const int pc = ctx - key0;     // tile column of tree node 0 (may be < 0 or >= 128)
                            const unsigned __int128 a128 =
                                ((unsigned __int128)(((unsigned long long)anc[3] << 32) | anc[2]) << 64) |
                                (unsigned __int128)(((unsigned long long)anc[1] << 32) | anc[0]);
                            unsigned __int128 vm;
                            if (pc >= 128) vm = ~(unsigned __int128)0;
                            else if (pc > 0) vm = (((unsigned __int128)1 << pc) - 1) | (a128 << pc);
                            else if (pc > -128) vm = a128 >> (-pc);
                            else vm = 0;
                            const uint32_t vw[4] = {(uint32_t)vm, (uint32_t)(vm >> 32), (uint32_t)(vm >> 64), (uint32_t)(vm >> 96)};
#pragma unroll
                            for (int c = 0; c < 128; ++c)
                                v[c] = ((vw[c >> 5] >> (c & 31)) & 1u) ? v[c] : 0xFF800000u;   // -inf
                        }
                        // one warp per scheduler: nothing hides a serial chain, so the row maximum (and the row
                        // sum below) run as four independent chains
                        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                        for (int c = 0; c < 128; c += 4) {
                            mx4[0] = fmaxf(mx4[0], __uint_as_float(v[c]));     mx4[1] = fmaxf(mx4[1], __uint_as_float(v[c + 1]));
                            mx4[2] = fmaxf(mx4[2], __uint_as_float(v[c + 2])); mx4[3] = fmaxf(mx4[3], __uint_as_float(v[c + 3]));
                        }
                        float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                        mx *= scale_log2;                  // scale > 0
                        const float m_new = fmaxf(m_run, mx);
                        // lazy rescaling: keep the stale maximum unless it grew by more than the threshold
                        const bool need = first ? true : (m_new > m_run + kRescaleThreshold);
                        if (__any_sync(0xFFFFFFFFu, need)) {
                            const float alpha = (m_run == -INFINITY) ? 0.f : ex2(m_run - m_new);
                            if (!first) {
                                // O holds tiles < t of this segment: wait for PV(t-1), then scale the row
                                ok = mbar_wait(hd, &hd->pv_done, (jg - 1) & 1, status);
                                if (ok) {
                                    tc_fence_after();
                                    uint32_t o[32];
                                    const uint32_t o_addr = tmem + kColO + lane_sel;
#pragma unroll
                                    for (int cc = 0; cc < 4; ++cc) {
                                        TMEM_LD32(o_addr + cc * 32, o, 0);
                                        tmem_wait_ld();
#pragma unroll
                                        for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
                                        TMEM_ST32(o_addr + cc * 32, o, 0);
                                    }
                                    tmem_wait_st();
                                }
                            }
                            l_run *= alpha;
                            m_run = m_new;
                        }
                        m_use = (m_run == -INFINITY) ? 0.f : m_run;
                    }
                    // P (bf16 pairs) overwrites the first 64 columns of this tile's S buffer: this thread has its whole
                    // S row in registers, and QK^T of tile jg+2 is ordered after PV(jg) in the MMA pipe
                    if (warp_has_rows) {
                        float ls4[4] = {0.f, 0.f, 0.f, 0.f};
                        const float neg_m = -m_use;
#pragma unroll
                        for (int e = 0; e < 64; ++e) {
                            float p0 = ex2(fmaf(__uint_as_float(v[2 * e]), scale_log2, neg_m));
                            float p1 = ex2(fmaf(__uint_as_float(v[2 * e + 1]), scale_log2, neg_m));
                            ls4[e & 3] += p0 + p1;
                            v[e] = pack_bf16x2(p0, p1);
                        }
                        l_run += (ls4[0] + ls4[1]) + (ls4[2] + ls4[3]);
                        const uint32_t p_taddr = tmem + kColS + (jg & 1) * 128 + lane_sel;
                        TMEM_ST32(p_taddr, v, 0);
                        TMEM_ST32(p_taddr + 32, v, 32);
                        tmem_wait_st();
                    }
                    // observe every phase of pv_done in order (a parity wait must never lag two phases behind its
                    // barrier); by now PV(jg-1) has normally completed, so this does not stall
                    if (jg > 0) ok = mbar_wait(hd, &hd->pv_done, (jg - 1) & 1, status);
                    if (!ok) break;
                    // ragged end: V rows past the sequence's last key may hold anything -> zero them
                    if ((t + 1) * kTile > n_keys) {
                        const uint32_t ring = 2 * jg + 1, st = ring % kStages;
                        ok = mbar_wait(hd, &hd->kv_full[st], (ring / kStages) & 1, status);
                        if (!ok) break;
                        const int r_local = sm_tid;        // one V row (key) per thread
                        if (t * kTile + r_local >= n_keys) {
                            unsigned char* vrow = kv_smem + st * kStageBytes + r_local * 128;
#pragma unroll
                            for (int c = 0; c < 8; ++c) {
                                *reinterpret_cast<uint4*>(vrow + c * 16) = make_uint4(0, 0, 0, 0);
                                *reinterpret_cast<uint4*>(vrow + kHalfBytes + c * 16) = make_uint4(0, 0, 0, 0);
                            }
                        }
                        fence_proxy_async();               // generic-proxy writes -> visible to the tensor core
                    }
                    tc_fence_before();
                    mbar_arrive(&hd->p_ready);
                    ++jg;
                    ++seg_tiles;
                    cu.next(wk);
                }
                if (!ok) break;

                // ---------------- segment epilogue: O of tiles [t_first, t_last] is complete after PV(jg-1)
                ok = mbar_wait(hd, &hd->pv_done, (jg - 1) & 1, status);
                if (!ok) break;
                tc_fence_after();
                const int n_tiles_seg = seg_tiles;
                const bool whole_head = (t_first == 0) && (n_tiles_seg == T);
                if (warp_has_rows) {
                    const uint32_t o_addr = tmem + kColO + lane_sel;
                    TMEM_LD32(o_addr, v, 0); TMEM_LD32(o_addr + 32, v, 32);
                    TMEM_LD32(o_addr + 64, v, 64); TMEM_LD32(o_addr + 96, v, 96);
                    tmem_wait_ld();
                }
                tc_fence_before();
                mbar_arrive(&hd->o_free);                  // TMEM O may be overwritten by the next segment

                const int hq = hk * g + member;            // query head of this row
                if (whole_head) {
                    if (row_valid) {
                        const float inv = bad ? 0.f : 1.f / l_run;
                        uint4* dst = reinterpret_cast<uint4*>(out + (((size_t)s0 * B + node) * H + hq) * kHeadDim);
#pragma unroll
                        for (int ch = 0; ch < 16; ++ch) {
                            uint32_t pk[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                pk[e] = bad ? 0u : pack_bf16x2(__uint_as_float(v[ch * 8 + 2 * e]) * inv,
                                                               __uint_as_float(v[ch * 8 + 2 * e + 1]) * inv);
                            dst[ch] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        }
                        if (lse) lse[((size_t)s0 * B + node) * H + hq] = bad ? 0.f : (m_run + log2f(l_run)) * kLn2;
                    }
                } else {
                    // partial -> workspace slot of this CTA (combined by tree_attn_combine_kernel): O/l in fp16
                    // (relative error 2^-11, far below the bf16 rounding of the final output), m and l in fp32
                    const int slot = 2 * blockIdx.x + (t_first == 0 ? 1 : 0);
                    float* part = partials + (size_t)slot * kUmmaPartFloats;
                    if (row_valid) {
                        // invalid parent[]: a neutral partial (O = 0; the head's first part carries weight 1)
                        // makes the combine kernel produce the defined zero output without re-validating
                        const float inv = (bad || l_run == 0.f) ? 0.f : 1.f / l_run;
                        uint4* dst = reinterpret_cast<uint4*>(part) + row;
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            uint32_t hw[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                __half2 h2 = __floats2half2_rn(__uint_as_float(v[8 * c + 2 * e]) * inv,
                                                               __uint_as_float(v[8 * c + 2 * e + 1]) * inv);
                                hw[e] = *reinterpret_cast<uint32_t*>(&h2);
                            }
                            dst[c * 128] = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                        }
                        part[kPartHalfWords + row] = bad ? (t_first == 0 ? 0.f : -INFINITY) : m_run;
                        part[kPartHalfWords + kMaxB + row] = bad ? (t_first == 0 ? 1.f : 0.f) : l_run;
                    }
                }
                ++seg;
            }
        }
    }

    // ---- teardown
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 queries [rows][Hkv][g][128] -> 4-D map, box = 64 x g x 1 x box_rows: the g query heads of one key/value
// head for box_rows consecutive nodes, landing as rows (node, member) of one 128-byte-swizzled tile
bool make_q_map(void* fn, CUtensorMap* map, const void* base, int64_t rows, int Hkv, int g, int box_rows) {
    cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)g, (cuuint64_t)Hkv, (cuuint64_t)rows};
    cuuint64_t strides[3] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)g * kHeadDim * 2, (cuuint64_t)Hkv * g * kHeadDim * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)g, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base),
                                                     dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// bf16 tensor [rows][H][128] -> 3-D map, box = 64 x 1 x box_rows, 128-byte swizzle, zero fill out of bounds
bool make_map(void* fn, CUtensorMap* map, const void* base, int64_t rows, int H, int box_rows) {
    cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)H, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)H * kHeadDim * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base),
                                                     dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace

// Self-test of the bounded-wait path: one warp waits on a barrier that nothing ever completes, with a short
// limit.  The wait must give up, set GOOSE_ST_TIMEOUT in status[0] and let the kernel return normally, the same way
// a stalled pipeline of the attention kernel would.  Nothing here can hang: the only loop is the bounded wait.
__global__ void __launch_bounds__(32)
bounded_wait_selftest_kernel(int32_t* __restrict__ status, long long limit_cycles, int32_t* __restrict__ result) {
    __shared__ Header hd;
    if (threadIdx.x == 0) {
        mbar_init(&hd.pv_done, 1);
        hd.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    bool ok = true;
    if (threadIdx.x == 0) ok = mbar_wait_limit(&hd, &hd.pv_done, 0, status, limit_cycles);   // never completes
    __syncwarp();
    // the other lanes see the abort flag at once, as the other roles of the attention kernel would
    if (threadIdx.x != 0) ok = mbar_wait_limit(&hd, &hd.pv_done, 0, status, limit_cycles);
    // the shared primitive the top-k kernel waits with: 1 (aborted) with the raised flag, 2 (timed out) with a clear one
    __shared__ volatile int no_flag;
    if (threadIdx.x == 1) no_flag = 0;
    __syncwarp();
    int bad = 0;
    if (threadIdx.x == 1) {
        bad |= mbar_wait_bounded(&hd.pv_done, 0, limit_cycles, &hd.abort_flag) != 1;
        bad |= mbar_wait_bounded(&hd.pv_done, 0, limit_cycles, &no_flag) != 2;
        result[0] = (ok ? 1 : 0) | (bad ? 2 : 0);          // 0 expected: every wait reported failure, the kernel returns
    }
}

cudaError_t launch_bounded_wait_selftest(goose_ctx* c, long long limit_cycles, int32_t* result, cudaStream_t st) {
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(c->status, limit_cycles, result);
    c->launches++;
    return cudaGetLastError();
}

cudaError_t init_umma_kernel() {
    cudaError_t e = cudaFuncSetAttribute(tree_attn_umma_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(tree_attn_umma_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(tree_attn_umma_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(tree_attn_umma_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmem);
}

int auto_attn_impl(const goose_ctx* c, int S, int B, int H) {
    (void)S; (void)H;
    (void)B;
    // the tcgen05 kernel wins at every tree size measured (B = 16: 15.8 us vs 31 us on the tiny workload);
    // the mma.sync kernel remains as the path for drivers that cannot encode tensor maps and on request
    return c->encode_tiled ? GOOSE_ATTN_UMMA : GOOSE_ATTN_MMA;
}

cudaError_t launch_tree_attn_umma(goose_ctx* c, const __nv_bfloat16* q, const __nv_bfloat16* kc,
                                  const __nv_bfloat16* vc, int64_t kv_rows, const int64_t* row_off,
                                  const int32_t* ctx_len, const int32_t* parent, const int32_t* n_nodes, int S, int B, int H,
                                  int Hkv, float scale, __nv_bfloat16* out, float* lse, cudaStream_t st,
                                  CombinePlan* defer_merge) {
    if (defer_merge) defer_merge->valid = false;
    if (!c->encode_tiled) return cudaErrorNotSupported;
    if (S == 0) return cudaSuccess;
    const int g = H / Hkv;                              // query heads per key/value head (validated by the caller)
    const int nb = B * g <= kTile ? B : kTile / g;      // nodes per M tile
    const int n_mt = (B + nb - 1) / nb;
    CUtensorMap mq, mk, mv;
    if (!make_q_map(c->encode_tiled, &mq, q, (int64_t)S * B, Hkv, g, nb) ||
        !make_map(c->encode_tiled, &mk, kc, kv_rows, Hkv, kTile) ||
        !make_map(c->encode_tiled, &mv, vc, kv_rows, Hkv, kTile))
        return cudaErrorInvalidValue;
    int grid = c->num_sms;
    if (2 * grid > c->n_slots) grid = c->n_slots / 2;
    const bool grouped = g > 1;
    const bool counts = n_nodes != nullptr;
    auto main_kernel = grouped ? (counts ? tree_attn_umma_kernel<true, true> : tree_attn_umma_kernel<true, false>)
                               : (counts ? tree_attn_umma_kernel<false, true> : tree_attn_umma_kernel<false, false>);
    cudaError_t e = launch_pdl(main_kernel, dim3(grid),
                               dim3(kThreads), kUmmaSmem, st, mq, mk, mv, row_off, ctx_len, parent, n_nodes, S, B, H, Hkv, g, nb,
                               kv_rows, scale * kLog2e, c->partials, c->status, out, lse);
    c->launches++;
    if (e != cudaSuccess) return e;
    CombineArgs ca;
    ca.ctx_len = ctx_len; ca.n_nodes = n_nodes; ca.S = S; ca.B = B; ca.H = H; ca.Hkv = Hkv; ca.g = g; ca.nb = nb;
    ca.G = grid; ca.Hw = n_mt * Hkv; ca.partials = c->partials; ca.out = out; ca.lse = lse;
    const int row_groups = (nb * g + 31) / 32;
    if (defer_merge) {                                  // the caller runs the merge as a role of a later launch
        defer_merge->args = ca; defer_merge->row_groups = row_groups; defer_merge->grouped = grouped;
        defer_merge->valid = true;
        return cudaSuccess;
    }
    auto merge_kernel = grouped ? (counts ? tree_attn_combine_kernel<true, true> : tree_attn_combine_kernel<true, false>)
                                : (counts ? tree_attn_combine_kernel<false, true> : tree_attn_combine_kernel<false, false>);
    e = launch_pdl(merge_kernel, dim3(row_groups, ca.Hw, S), dim3(kCombineThreads), 0, st, ca);
    c->launches++;
    return e;
}

}  // namespace goose
