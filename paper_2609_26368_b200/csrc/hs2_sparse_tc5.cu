// Sparse attention over idx ∪ window for large head groups on the 5th-generation tensor cores
// (Section 3.3: the sparse layers attend to the selected tokens plus the sliding window; Table 1: the
// paper's own models share one KV head among 64 query heads of dimension 256).
//
// With G = 64 heads per KV head every gathered key row is used by 64 heads, i.e. 64 flop per byte: the
// gather tile is a dense contraction and belongs on tcgen05.  Work item = one (sequence, KV head, sub-group
// of up to 64 heads, query); persistent CTAs walk the items with all pipelines running across item boundaries.
//   rows of the MMA (M = 128, TMEM lane) = the heads of the item (lanes >= 64 hold don't-care rows),
//   columns = 64 gathered keys per tile.
//   gather warps  slot s of the virtual array [idx row | window] -> key index -> the key's K or V row copied
//              with 16-byte cp.async into the 128-byte-swizzled UMMA operand layout (void slots are zero
//              filled).  K and V have warp groups and rings of their own (K is released as soon as Q K^T has
//              read it, V after P V); completion reaches the mbarrier without blocking the thread
//              (cp.async.mbarrier.arrive).  The copy rate grows with the number of issuing warps, hence four
//              warps per group at head_dim 256.  Q (the item's heads) arrives by TMA.
//   MMA warp   S = Q K^T (M128 N64 K=D) into one of two TMEM buffers, O += P V (V as MN-major B operand).
//   softmax    four warps, two threads per head (32 keys of the tile each; the row maximum is exchanged through
//              shared memory): online softmax in the base-2 domain with a lazily rescaled accumulator as in
//              the full-attention kernel, void slots masked, optional sink logit in the denominator; P is
//              double buffered so that the exponentials of tile g+1 overlap P V of tile g.
// Every mbarrier wait is bounded; a wait that runs out sets a device error word, the CTA drains its copies,
// frees its TMEM and returns.
#include <cuda.h>

#include "hs2_common.cuh"
#include "hs2_tc5.cuh"

namespace hs2 {

__device__ unsigned g_sptc5_error;   // bit 0: an mbarrier wait ran out; bit 1: shared-memory base not alignable

namespace {

using namespace tc5;

constexpr int BM = 128, BN = 64;
// Warps per gather group at head_dim 256.  Measured on the paper's shape (64 heads, 1152 keys per query): 2 -> 2.17 ms,
// 3 -> 1.77 ms, 4 -> 1.60 ms, 5 -> 1.64 ms, 6 -> 2.28 ms (register cap forces spills).
#ifndef HS2_SP_PWARPS
#define HS2_SP_PWARPS 4
#endif
constexpr int kSubHeads = 64;              // heads per work item (a larger group is walked in sub-groups)
constexpr uint32_t kBarBytes = 256;
constexpr uint32_t kAlignSlack = 896;
constexpr float kRescaleThreshold = 8.f;   // log2 units

// Warp roles (the TMEM lanes 0-63 that hold the 64 heads are only reachable from warps with index % 4 in {0, 1}):
//   0, 1, 4, 5  softmax: warp & 1 = TMEM lane quadrant (heads 0-31 / 32-63), warp >> 2 = column half of the tile
//   2           MMA issuer (also owns the TMEM allocation)
//   3, 6, 7..   gather producers: the first PW of them copy K, the next PW copy V
__device__ __forceinline__ bool is_softmax_warp(int w) { return w < 6 && (w & 3) < 2; }
__device__ __forceinline__ int producer_ordinal(int w) { return w == 3 ? 0 : w - 5; }

// Shared-memory plan for head_dim D.  The MMA always reads 128 A rows per 64-dim slice of Q; rows past the 64
// that are loaded alias whatever follows (the next slice or the K ring), which is harmless: they only produce
// TMEM lanes that nobody reads.
#ifndef HS2_SPTC5_PTMEM
#define HS2_SPTC5_PTMEM 1   // P as a tensor-memory operand of P V (0: through shared memory)
#endif
#ifndef HS2_SPTC5_CLUSTER
#define HS2_SPTC5_CLUSTER 1   // split queries merge inside a thread-block cluster (0: through scratch and a second kernel)
#endif
#ifndef HS2_SPTC5_VST3
#define HS2_SPTC5_VST3 1    // three V stages at head_dim 256 (needs P in tensor memory)
#endif

// F8: the cache holds e4m3 codes with one fp32 scale per (token, KV head); the gather warps dequantise the codes into
// the bf16 operand layout, the softmax applies the scales (see the kernel).
template <int D, bool F8 = false>
struct SpCfg {
    static constexpr int NQ = D / 64;                           // 64-dim slices of an operand tile
    static constexpr int CH = D / 8;                            // 16-byte chunks per row
    static constexpr int KST = D == 256 ? 3 : 2;                // K ring depth
    // V ring depth: with P in tensor memory its 16 KB of shared memory, and most of the alignment slack, buy a third
    // V stage at head_dim 256 (the layout then fills the 227 KB to the byte)
    static constexpr int VST = (D == 256 && HS2_SPTC5_PTMEM && HS2_SPTC5_VST3 && !F8) ? 3 : 2;   // (the FP8 variant's register loads need the room less)
    static constexpr uint32_t kSlack = VST == 3 ? 256 : kAlignSlack;
    static constexpr int PW = D == 256 ? HS2_SP_PWARPS : 1;     // warps per gather group (one K group, one V group)
    static constexpr int kThreads = (5 + 2 * PW) * 32;
    static constexpr uint32_t kQSlice = kSubHeads * 128;
    static constexpr uint32_t kQBytes = NQ * kQSlice;
    static constexpr uint32_t kKVStage = NQ * BN * 128;
    static constexpr uint32_t kOffQ = 0;
    // two P buffers of 64 real rows x 64 keys bf16, 8 KB apart; the 128 rows the MMA reads from the second one run
    // on into the K ring (don't-care rows again)
    static constexpr uint32_t kOffP = kOffQ + kQBytes;
    static constexpr uint32_t kPStride = kSubHeads * 128;
    static constexpr uint32_t kOffK = kOffP + (HS2_SPTC5_PTMEM ? 0 : 2 * kPStride);
    static constexpr uint32_t kOffV = kOffK + KST * kKVStage;
    static constexpr uint32_t kOffKey = kOffV + VST * kKVStage;   // int[2 groups][2][64]: key index per slot of a tile
    static constexpr uint32_t kOffMx = kOffKey + 4 * BN * 4;    // float[2 tiles][2 halves][64]: row maxima exchanged
    static constexpr uint32_t kOffL = kOffMx + 4 * 64 * 4;      // float[2 halves][64]: row sums exchanged
    static constexpr uint32_t kOffSc = kOffL + 2 * 64 * 4;      // FP8: float[4 softmax warps][K scale, V scale][32 keys]
    static constexpr uint32_t kOffBar = kOffSc + (F8 ? 4 * 2 * 32 * 4 : 0);
    static constexpr uint32_t kSmemBytes = kOffBar + kBarBytes + kSlack;
    // cluster merge: a CTA's unnormalised partial (64 rows of D floats, 16 bytes of padding per row, then maximum and
    // sum per row) lies in its K/V rings, which are idle by then
    static constexpr uint32_t kPartPitch = (D + 4) * 4;
    static constexpr uint32_t kOffPartMl = kOffK + kSubHeads * kPartPitch;
    static_assert(kOffPartMl + kSubHeads * 8 <= kOffKey, "the partial fits the K and V rings");
    static constexpr uint32_t kTmem = D <= 128 ? 256 : 512;     // 2 x 64 score columns + D output columns
    static constexpr int kMinBlocks = D <= 128 ? 2 : 1;
    static_assert(kOffQ + (NQ - 1) * kQSlice + BM * 128 <= kOffKey && (HS2_SPTC5_PTMEM || kOffP + kPStride + BM * 128 <= kOffKey),
                  "the 128 A rows the MMA reads stay inside the buffer");
    static_assert(kSmemBytes <= 227 * 1024, "fits the shared memory of one SM");
};

enum Bar {
    Q_FULL = 0, Q_EMPTY, K_FULL0, K_FULL1, K_FULL2, K_EMPTY0, K_EMPTY1, K_EMPTY2, V_FULL0, V_FULL1, V_FULL2, V_EMPTY0, V_EMPTY1, V_EMPTY2,
    S_FULL0, S_FULL1, S_FREE0, S_FREE1, P_FULL0, P_FULL1, PV_DONE0, PV_DONE1, O_FREE, N_BARS
};
static_assert(N_BARS * 8 + 8 <= kBarBytes, "barriers, TMEM slot and abort flag fit their block");

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    return tc5::mbar_wait(bar, parity, abort_flag, &g_sptc5_error);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes)
{
    // .ca: measured a little faster than .cg here (the rows of a tile are touched once either way)
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// the mbarrier receives one arrival from this thread once all its earlier cp.async copies have landed
__device__ __forceinline__ void cp_async_arrive(uint32_t bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;\n" ::: "memory"); }
// ---- thread-block clusters: the CTAs that share one query's keys merge their partial results through each other's
// ---- shared memory (plain loads from a peer's window; no multicast anywhere)
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ uint32_t peer_smem(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 ld_peer4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float2 ld_peer2(uint32_t addr)
{
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];\n" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
    return v;
}

// two e4m3 codes (low byte first) -> two bf16 (exact: e4m3 has 3 mantissa bits and a range bf16 covers)
__device__ __forceinline__ uint32_t e4m3x2_to_bf16x2(uint32_t two_codes)
{
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;\n" : "=r"(h2) : "h"((unsigned short)two_codes));
    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
    return pack_bf16(f.x, f.y);
}
__device__ __forceinline__ uint4 ld_codes16(const char *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Slot s of the virtual slot array [idx row | window] of a query at position pos holds a key index or is void (-1).
// slot_raw starts the fetch (an idx entry is a global load) and slot_fix applies the validity rules to it; callers
// keep the raw value in a register for a whole tile so that the load's latency is never waited for.
__device__ __forceinline__ int slot_raw(const Params &p, const int32_t *irow, int pos, int s)
{
    if (s < p.k) return irow ? __ldg(irow + s) : -1;
    return s < p.k + p.w ? pos - p.w + 1 + (s - p.k) : -1;
}
__device__ __forceinline__ int slot_fix(const Params &p, int j, int pos, int kvl, int s)
{
    const int hi = s < p.k ? pos - p.w : pos;   // idx entries inside the window are void: the window slots cover them
    return (j < 0 || j > hi || j >= kvl) ? -1 : j;
}

// Persistent: every CTA walks items blockIdx.x, blockIdx.x + gridDim.x, ...  All rings and phases are indexed by
// the running tile number g = (items done by this CTA) * nblk + t, which every role computes for itself.
// With n_splits > 1 (few queries, e.g. decode) an item is one of n_splits runs of nblk tiles of a query's slot
// array (slots past the array are void), and it leaves an unnormalised partial (running maximum, sum, fp32
// accumulator) in part_ml / part_o for the combine kernel below - or, when part_o is null, the n_splits CTAs of a
// query are one thread-block cluster (launched so: the grid is exactly the items, the cluster is the query) and merge
// through distributed shared memory: every CTA parks its partial in its own, by then idle, K/V rings, and after a
// cluster barrier CTA c reads column slice c of every peer's partial, merges and stores it.  No scratch, one launch.
template <int D, bool F8>
__global__ void __launch_bounds__(SpCfg<D, F8>::kThreads, SpCfg<D, F8>::kMinBlocks)
k_sparse_tc5(const __grid_constant__ CUtensorMap tmQ, const Params p, const void *__restrict__ K,
             const void *__restrict__ V, const float *__restrict__ ksc, const float *__restrict__ vsc,
             const int32_t *__restrict__ idx, const float *__restrict__ sink,
             __nv_bfloat16 *__restrict__ O, float *__restrict__ LSE, int64_t n_items, int n_sub, int n_splits, int nblk,
             float *__restrict__ part_ml, float *__restrict__ part_o)
{
    using C = SpCfg<D, F8>;
    constexpr int NQ = C::NQ, CH = C::CH, KST = C::KST;
    constexpr uint32_t kKVStage = C::kKVStage;
    extern __shared__ char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    if (pad > C::kSlack) {
        if (threadIdx.x == 0) atomicOr(&g_sptc5_error, 2u);
        return;
    }
    char *smem = smem_raw + pad;
    const uint32_t sbase = raw + pad;
    const uint32_t bars = sbase + C::kOffBar;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::kOffBar + N_BARS * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::kOffBar + N_BARS * 8 + 4);
    int *s_key = reinterpret_cast<int *>(smem + C::kOffKey);
    float *s_mx = reinterpret_cast<float *>(smem + C::kOffMx);
    float *s_l = reinterpret_cast<float *>(smem + C::kOffL);
    auto bar = [&](int i) { return bars + 8u * i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // item -> (sequence, KV head, sub-group of heads, query, position)
    struct Where { int b, gkv, sub, i, kvl, pos, slot0; };
    auto where = [&](int64_t item) {
        Where wq;
        wq.slot0 = (int)(item % n_splits) * nblk * BN;   // first slot of this run of tiles
        item /= n_splits;
        wq.i = (int)(item % p.Lq);
        const int r = (int)(item / p.Lq);
        wq.sub = r % n_sub;
        const int bg = r / n_sub;
        wq.gkv = bg % p.Hkv;
        wq.b = bg / p.Hkv;
        wq.kvl = kvlen_of(p, wq.b);
        wq.pos = pos_of(p, wq.b, wq.i);
        return wq;
    };
    auto irow_of = [&](const Where &wq) {
        return (p.k > 0 && idx) ? idx + (((int64_t)wq.b * p.Hkv + wq.gkv) * p.Lq + wq.i) * p.k : (const int32_t *)nullptr;
    };
    const int box_heads = p.G < kSubHeads ? p.G : kSubHeads;

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(Q_FULL), 1); mbar_init(bar(Q_EMPTY), 1);
        for (int s = 0; s < 3; ++s) {
            mbar_init(bar(K_FULL0 + s), 32 * C::PW); mbar_init(bar(K_EMPTY0 + s), 1);
            mbar_init(bar(V_FULL0 + s), 32 * C::PW); mbar_init(bar(V_EMPTY0 + s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(S_FULL0 + s), 1); mbar_init(bar(S_FREE0 + s), 128);
            mbar_init(bar(P_FULL0 + s), 128); mbar_init(bar(PV_DONE0 + s), 1);
        }
        mbar_init(bar(O_FREE), 128);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(C::kTmem) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (is_softmax_warp(warp)) {
        // ------------------------------------------------ softmax: two threads per head, 32 keys of a tile each
        // Every thread of a quadrant pair executes the same sequence of pair barriers; a wait that runs out only
        // marks the thread dead, and the next pair barrier then ends both loops together.
        const int quad = warp & 1, half = warp >> 2;
        const int row = 32 * quad + lane;
        const int pair_bar = 3 + quad;
        const uint32_t lane_base = tmem + ((uint32_t)(32 * quad) << 16);
        const uint32_t o_col0 = 2 * BN + half * (D / 2);    // this thread's half of the output columns
        bool alive = true, dead = false;
        int n = 0;
        for (int64_t item = blockIdx.x; item < n_items && alive; item += gridDim.x, ++n) {
            const Where q = where(item);
            const bool real = row < min(kSubHeads, p.G - kSubHeads * q.sub);
            const int h = q.gkv * p.G + kSubHeads * q.sub + (real ? row : 0);
            const int32_t *irow = irow_of(q);
            float m_used = -INFINITY, l = 0.f;
            if (sink && real && q.slot0 == 0) {   // Section 3.3 variant with a learnable sink logit: it only joins the denominator
                m_used = sink[h] * kLog2e;
                l = half == 0 ? 1.f : 0.f;
            }
            const int g0 = n * nblk;
            // validity of this half's 32 slots is recomputed here (cheap, and no cross-warp visibility to argue
            // about), one tile ahead so that the idx loads are off the critical path
            const int my_slot = q.slot0 + 32 * half + lane;
            int jn = slot_raw(p, irow, q.pos, my_slot);
            // FP8 cache: this lane's slot also tells it which key's scales the tile needs.  The key index is kept a tile
            // further ahead (jn2) so that the scales of tile t+1 can be requested while tile t is worked on; they
            // reach the other threads of the warp through a warp-private patch of shared memory.
            float ks_cur = 0.f, vs_cur = 0.f;
            int jn2 = -1;
            float *my_sc = reinterpret_cast<float *>(smem + C::kOffSc) + ((warp & 1) + 2 * (warp >> 2)) * 64;
            if (F8) {
                const int j0 = slot_fix(p, jn, q.pos, q.kvl, my_slot);
                if (j0 >= 0) {
                    const int64_t so = q.b * p.ss_b + (int64_t)j0 * p.ss_t + q.gkv * p.ss_h;
                    ks_cur = __ldg(ksc + so);
                    vs_cur = __ldg(vsc + so);
                }
                if (nblk > 1) jn2 = slot_raw(p, irow, q.pos, my_slot + BN);
            }
            for (int t = 0; t < nblk; ++t) {
                const int g = g0 + t, sb = g & 1;
                const uint32_t valid = __ballot_sync(0xffffffffu, slot_fix(p, jn, q.pos, q.kvl, my_slot + t * BN) >= 0);
                if (!F8) {
                    if (t + 1 < nblk) jn = slot_raw(p, irow, q.pos, my_slot + (t + 1) * BN);
                } else {
                    __syncwarp();   // the previous tile's scales have been read by every lane
                    my_sc[lane] = ks_cur;
                    my_sc[32 + lane] = vs_cur;
                    jn = jn2;       // raw entry of tile t+1, fetched a tile ago
                    ks_cur = 0.f; vs_cur = 0.f;
                    if (t + 1 < nblk) {
                        const int j1 = slot_fix(p, jn, q.pos, q.kvl, my_slot + (t + 1) * BN);
                        if (j1 >= 0) {
                            const int64_t so = q.b * p.ss_b + (int64_t)j1 * p.ss_t + q.gkv * p.ss_h;
                            ks_cur = __ldg(ksc + so);
                            vs_cur = __ldg(vsc + so);
                        }
                        if (t + 2 < nblk) jn2 = slot_raw(p, irow, q.pos, my_slot + (t + 2) * BN);
                    }
                    __syncwarp();
                }
                if (!dead && !__all_sync(0xffffffffu, mbar_wait(bar(S_FULL0 + sb), (g >> 1) & 1, abort_flag))) dead = true;
                float s[32];
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
                if (!dead) {
                    tc_fence_after();
                    tmem_ld32(lane_base + sb * BN + 32 * half, s);
                    tmem_wait_ld();
                    tc_fence_before();
                    mbar_arrive(bar(S_FREE0 + sb));
                    if (F8) {   // the K scale of a key multiplies its score (void slots: 0 * 0, masked below)
#pragma unroll
                        for (int e4 = 0; e4 < 32; e4 += 4) {
                            const float4 kq = *reinterpret_cast<const float4 *>(my_sc + e4);
                            s[e4] *= kq.x; s[e4 + 1] *= kq.y; s[e4 + 2] *= kq.z; s[e4 + 3] *= kq.w;
                        }
                    }
                    if (valid != 0xffffffffu) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (!((valid >> e) & 1u)) s[e] = -INFINITY;
                    }
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        mx0 = fmaxf(mx0, s[e]); mx1 = fmaxf(mx1, s[e + 1]); mx2 = fmaxf(mx2, s[e + 2]); mx3 = fmaxf(mx3, s[e + 3]);
                    }
                }
                float m_raw = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                s_mx[((g & 1) * 2 + half) * 64 + row] = m_raw;
                if (!group_all(pair_bar, 64, !dead)) { alive = false; break; }
                m_raw = fmaxf(m_raw, s_mx[((g & 1) * 2 + (half ^ 1)) * 64 + row]);
                const float m_blk = m_raw * p.scale_log2;
                const bool need = m_blk > m_used + kRescaleThreshold;
                const float m_new = need ? m_blk : m_used;
                const float corr = need ? exp2f(m_used - m_new) : 1.f;
                // P V of tile g-2 has read the P buffer this tile writes (two buffers, two barriers: a barrier's next
                // completion always depends on this thread, so a parity wait can never be a phase behind)
                if (g > 1 && !dead && !__all_sync(0xffffffffu, mbar_wait(bar(PV_DONE0 + sb), ((g - 2) >> 1) & 1, abort_flag))) dead = true;
                if (t > 0 && __any_sync(0xffffffffu, need)) {   // rare: rescale the accumulator, after P V of tile g-1
                    if (!dead && !__all_sync(0xffffffffu, mbar_wait(bar(PV_DONE0 + (sb ^ 1)), ((g - 1) >> 1) & 1, abort_flag))) dead = true;
                    if (!dead) {
                        tc_fence_after();
#pragma unroll
                        for (int cc = 0; cc < D / 64; ++cc) {
                            float o[32];
                            tmem_ld32(lane_base + o_col0 + cc * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] *= corr;
                            tmem_st32(lane_base + o_col0 + cc * 32, o);
                        }
                        tmem_wait_st();
                    }
                }
                l *= corr;
                m_used = m_new;
                if (!dead) {
                    const float neg_m = m_used == -INFINITY ? 0.f : -m_used;
                    uint32_t pk[16];
                    float l0 = 0.f, l1 = 0.f;
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const float p0 = exp2f(fmaf(s[e], p.scale_log2, neg_m));       // -inf stays -inf -> 0
                        const float p1 = exp2f(fmaf(s[e + 1], p.scale_log2, neg_m));
                        l0 += p0; l1 += p1;
                        if (F8) {   // the V scale of a key rides on its probability into P V; the row sum stays unscaled
                            const float2 vq = *reinterpret_cast<const float2 *>(my_sc + 32 + e);
                            pk[e >> 1] = pack_bf16(p0 * vq.x, p1 * vq.y);
                        } else {
                            pk[e >> 1] = pack_bf16(p0, p1);
                        }
                    }
                    l += l0 + l1;
#if HS2_SPTC5_PTMEM
                    // P replaces the scores it came from: bf16 pairs over the first 32 columns of the score buffer, this
                    // half's 32 keys in 16 of them (the partner has read its scores: it passed the pair barrier above)
                    tmem_st16u(lane_base + sb * BN + 16 * half, pk);
                    tmem_wait_st();
#else
                    char *prow_ptr = smem + C::kOffP + sb * C::kPStride + row * 128;
#pragma unroll
                    for (int c4 = 0; c4 < 4; ++c4)   // 8 keys = one 16-byte chunk, chunk position XOR (row & 7)
                        *reinterpret_cast<uint4 *>(prow_ptr + (((half * 4 + c4) ^ (row & 7)) << 4)) =
                            make_uint4(pk[4 * c4], pk[4 * c4 + 1], pk[4 * c4 + 2], pk[4 * c4 + 3]);
                    fence_proxy_async();
#endif
                    tc_fence_before();
                    mbar_arrive(bar(P_FULL0 + sb));
                }
            }
            if (!alive) break;
            // ---- epilogue of the item: both P V barriers (every completion is observed, none can lap a wait)
            {
                const int gl = g0 + nblk - 1;
                if (!dead && gl > 0 && !__all_sync(0xffffffffu, mbar_wait(bar(PV_DONE0 + ((gl - 1) & 1)), ((gl - 1) >> 1) & 1, abort_flag))) dead = true;
                if (!dead && !__all_sync(0xffffffffu, mbar_wait(bar(PV_DONE0 + (gl & 1)), (gl >> 1) & 1, abort_flag))) dead = true;
            }
            s_l[half * 64 + row] = l;
            if (!group_all(pair_bar, 64, !dead)) { alive = false; break; }
            l += s_l[(half ^ 1) * 64 + row];
            tc_fence_after();
            const bool any = l > 0.f && m_used != -INFINITY;
            const float inv = any ? 1.f / l : 0.f;
            const int64_t o_off = q.b * p.os_b + (int64_t)q.i * p.os_t + h * p.os_h + half * (D / 2);
            __nv_bfloat16 *orow = O + o_off;
            const __nv_bfloat16 *grow = p.gate ? static_cast<const __nv_bfloat16 *>(p.gate) + o_off : nullptr;
            const bool by_cluster = n_splits > 1 && part_o == nullptr;
            float *prow = (n_splits > 1 && !by_cluster) ? part_o + (item * kSubHeads + row) * D + half * (D / 2) : nullptr;
            float *srow = reinterpret_cast<float *>(smem + C::kOffK + row * C::kPartPitch) + half * (D / 2);
#pragma unroll
            for (int cc = 0; cc < D / 64; ++cc) {
                float o[32];
                tmem_ld32(lane_base + o_col0 + cc * 32, o);
                tmem_wait_ld();
                if (cc == D / 64 - 1) {   // the accumulator may now be overwritten by the next item
                    tc_fence_before();
                    mbar_arrive(bar(O_FREE));
                }
                if (n_splits > 1) {   // unnormalised partial, every row (rows past the group are never combined)
                    float *dstp = by_cluster ? srow : prow;
#pragma unroll
                    for (int q4 = 0; q4 < 8; ++q4)
                        *reinterpret_cast<float4 *>(dstp + cc * 32 + q4 * 4) =
                            any ? make_float4(o[4 * q4], o[4 * q4 + 1], o[4 * q4 + 2], o[4 * q4 + 3]) : make_float4(0.f, 0.f, 0.f, 0.f);
                } else if (real) {
                    if (grow) {   // sigmoid output gate, before the single rounding to bf16
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const uint4 gv = *reinterpret_cast<const uint4 *>(grow + cc * 32 + q4 * 8);
                            const __nv_bfloat162 *gg = reinterpret_cast<const __nv_bfloat162 *>(&gv);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float2 g2 = __bfloat1622float2(gg[e]);
                                o[8 * q4 + 2 * e] *= gate_of(g2.x);
                                o[8 * q4 + 2 * e + 1] *= gate_of(g2.y);
                            }
                        }
                    }
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint4 v;
                        v.x = pack_bf16(o[8 * q4 + 0] * inv, o[8 * q4 + 1] * inv);
                        v.y = pack_bf16(o[8 * q4 + 2] * inv, o[8 * q4 + 3] * inv);
                        v.z = pack_bf16(o[8 * q4 + 4] * inv, o[8 * q4 + 5] * inv);
                        v.w = pack_bf16(o[8 * q4 + 6] * inv, o[8 * q4 + 7] * inv);
                        *reinterpret_cast<uint4 *>(orow + cc * 32 + q4 * 8) = v;
                    }
                }
            }
            if (n_splits > 1) {
                float *mlp = by_cluster ? reinterpret_cast<float *>(smem + C::kOffPartMl) + row * 2 : part_ml + (item * kSubHeads + row) * 2;
                if (half == 0) *reinterpret_cast<float2 *>(mlp) = make_float2(any ? m_used : -INFINITY, any ? l : 0.f);
            } else if (real && half == 0 && LSE) {
                LSE[((int64_t)q.b * p.Hq + h) * p.Lq + q.i] = any ? (m_used + log2f(l)) * kLn2 : -INFINITY;
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t idS = idesc(BM, BN, 0), idPV = idesc(BM, D, 1);
            const uint64_t dq = smem_desc(sbase + C::kOffQ, 16, 1024);
            bool ok = true;
            int n = 0;
            for (int64_t item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++n) {
                const int g0 = n * nblk;
                auto issue_s = [&](int t) -> bool {
                    const int g = g0 + t, ks = g % KST, sb = g & 1;
                    if (!mbar_wait(bar(K_FULL0 + ks), (g / KST) & 1, abort_flag)) return false;
                    if (!mbar_wait(bar(S_FREE0 + sb), ((g >> 1) & 1) ^ 1, abort_flag)) return false;
                    fence_proxy_async();   // the gathered rows were written through the generic proxy
                    tc_fence_after();
                    const uint64_t dk = smem_desc(sbase + C::kOffK + ks * kKVStage, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {   // descriptor address field counts 16-byte units
                        umma(tmem + sb * BN, dq + (((kk >> 2) * C::kQSlice + (kk & 3) * 32) >> 4),
                             dk + (((kk >> 2) * (BN * 128) + (kk & 3) * 32) >> 4), idS, kk > 0);
                    }
                    umma_commit(bar(S_FULL0 + sb));
                    umma_commit(bar(K_EMPTY0 + ks));
                    if (t == nblk - 1) umma_commit(bar(Q_EMPTY));
                    return true;
                };
                ok = mbar_wait(bar(Q_FULL), n & 1, abort_flag);
                ok = ok && issue_s(0);
                for (int t = 0; ok && t < nblk; ++t) {
                    if (t + 1 < nblk && !issue_s(t + 1)) { ok = false; break; }
                    const int g = g0 + t, pb = g & 1, vs = g % C::VST;   // P / score buffer, V stage
                    if (!mbar_wait(bar(P_FULL0 + pb), (g >> 1) & 1, abort_flag)) { ok = false; break; }
                    if (!mbar_wait(bar(V_FULL0 + vs), (g / C::VST) & 1, abort_flag) ||
                        (t == 0 && !mbar_wait(bar(O_FREE), (n & 1) ^ 1, abort_flag))) { ok = false; break; }
                    fence_proxy_async();
                    tc_fence_after();
#if !HS2_SPTC5_PTMEM
                    const uint64_t dp = smem_desc(sbase + C::kOffP + pb * C::kPStride, 16, 1024);
#endif
                    // V: MN-major B operand, 64-dim slices BN*128 bytes apart (leading offset), 8-key groups 1024 bytes apart
                    const uint64_t dv = smem_desc(sbase + C::kOffV + vs * kKVStage, BN * 128, 1024);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {   // 16 keys per instruction
#if HS2_SPTC5_PTMEM
                        // P: tensor-memory A operand, 16 keys = 8 columns of bf16 pairs; the in-order tensor pipe runs
                        // Q K^T of tile g+2, which overwrites that score buffer, after this instruction
                        umma_ts(tmem + 2 * BN, tmem + pb * BN + kk * 8, dv + ((kk * 2048) >> 4), idPV, (t > 0 || kk > 0) ? 1u : 0u);
#else
                        umma(tmem + 2 * BN, dp + ((kk * 32) >> 4), dv + ((kk * 2048) >> 4), idPV, (t > 0 || kk > 0) ? 1u : 0u);
#endif
                    }
                    umma_commit(bar(V_EMPTY0 + vs));
                    umma_commit(bar(PV_DONE0 + pb));
                }
            }
        }
    } else {
        // ------------------------------------------------ gather producers: a K group and a V group of PW warps
        // The groups run independently (own key records, own named barrier), so K can run KST tiles ahead of the
        // tensor core while V waits for P V to release its stage.
        // Thread -> one 16-byte chunk column c and every RPI-th row: a warp instruction copies whole key rows.
        constexpr int GT = 32 * C::PW;                // threads per group
        constexpr int RPI = GT / CH;                  // rows per iteration of the copy loop
        constexpr int KPT = (BN + GT - 1) / GT;       // key records per thread
        static_assert(GT % CH == 0, "a group's threads tile whole rows");
        const int po = producer_ordinal(warp);
        const int is_v = po / C::PW;
        const int gtid = (po % C::PW) * 32 + lane;
        const int c = gtid % CH, r0 = gtid / CH;
        const uint32_t dst_c = (uint32_t)(c >> 3) * (BN * 128);
        const int64_t row_bytes = p.ks_t * (F8 ? 1 : 2);
        const char *src_t = static_cast<const char *>(is_v ? V : K);
        // FP8: a thread takes one 16-byte run of codes (16 elements = two bf16 chunks) of every RPI8-th row
        constexpr int CH8 = D / 16, RPI8 = GT / CH8;
        const int c8 = gtid % CH8, r8 = gtid / CH8;
        const uint32_t ring0 = sbase + (is_v ? C::kOffV : C::kOffK) + dst_c;
        const int nst = is_v ? C::VST : KST;
        const int bar_full = is_v ? V_FULL0 : K_FULL0, bar_empty = is_v ? V_EMPTY0 : K_EMPTY0;
        int *keys_base = s_key + is_v * 2 * BN;       // two records per group
        // the key indices of a tile are fetched one tile ahead (the idx row is read from global memory, and that
        // latency would otherwise sit in front of every tile's copies; three and five tiles ahead measured the same)
        int j_next[KPT];
#pragma unroll
        for (int u = 0; u < KPT; ++u) j_next[u] = -1;
        if ((int64_t)blockIdx.x < n_items) {
            const Where q0 = where(blockIdx.x);
#pragma unroll
            for (int u = 0; u < KPT; ++u)
                if (gtid + u * GT < BN) j_next[u] = slot_raw(p, irow_of(q0), q0.pos, q0.slot0 + gtid + u * GT);
        }
        bool alive = true;
        int n = 0;
        for (int64_t item = blockIdx.x; item < n_items && alive; item += gridDim.x, ++n) {
            const Where q = where(item);
            const bool more = item + gridDim.x < n_items;
            const Where qn = where(more ? item + gridDim.x : item);
            const int32_t *irow = irow_of(q), *irow_n = irow_of(qn);
            const char *src0 = src_t + (q.b * p.ks_b + q.gkv * p.ks_h) * (F8 ? 1 : 2) + (F8 ? c8 : c) * 16;
            if (!is_v && gtid == 0) {   // Q of this item, once the last Q K^T of the previous item has read the buffer
                if (mbar_wait(bar(Q_EMPTY), (n & 1) ^ 1, abort_flag)) {
                    mbar_expect_tx(bar(Q_FULL), (uint32_t)(NQ * box_heads * 128));
#pragma unroll
                    for (int sl = 0; sl < NQ; ++sl)
                        tma_load_4d(sbase + C::kOffQ + sl * C::kQSlice, &tmQ, bar(Q_FULL), 64 * sl, q.gkv * p.G + kSubHeads * q.sub, q.i, q.b);
                }
            }
            for (int t = 0; t < nblk; ++t) {
                const int g = n * nblk + t;
                const int st = g % nst;
                int *keys = keys_base + (g & 1) * BN;   // double buffered: a thread is at most one barrier ahead
                int j_mine[KPT];
#pragma unroll
                for (int u = 0; u < KPT; ++u) {
                    const int sl = gtid + u * GT;
                    j_mine[u] = slot_fix(p, j_next[u], q.pos, q.kvl, q.slot0 + t * BN + sl);
                    if (sl < BN) {
                        if (t + 1 < nblk) j_next[u] = slot_raw(p, irow, q.pos, q.slot0 + (t + 1) * BN + sl);
                        else if (more) j_next[u] = slot_raw(p, irow_n, qn.pos, qn.slot0 + sl);
                    }
                }
                const bool ok = __all_sync(0xffffffffu, mbar_wait(bar(bar_empty + st), ((g / nst) & 1) ^ 1, abort_flag));
#pragma unroll
                for (int u = 0; u < KPT; ++u)
                    if (gtid + u * GT < BN) keys[gtid + u * GT] = j_mine[u];
                if (!group_all(1 + is_v, GT, ok)) { alive = false; break; }   // also publishes the key indices
                if (!F8) {
                    const uint32_t dst0 = ring0 + st * kKVStage;
#pragma unroll 4
                    for (int r = r0; r < BN; r += RPI) {
                        const int j = keys[r];
                        cp_async16(dst0 + r * 128 + (((c & 7) ^ (r & 7)) << 4), src0 + (j >= 0 ? (int64_t)j * row_bytes : 0), j >= 0 ? 16 : 0);
                    }
                    cp_async_arrive(bar(bar_full + st));
                } else {
                    // codes -> registers (eight rows in flight per thread) -> bf16 -> the two 16-byte chunks of the
                    // swizzled operand row; void slots are written as zeros
                    const uint32_t dst8 = sbase + (is_v ? C::kOffV : C::kOffK) + st * kKVStage + (uint32_t)(c8 >> 2) * (BN * 128);
                    constexpr int NIT = BN / RPI8, BATCH = NIT < 8 ? NIT : 8;
#pragma unroll 1
                    for (int i0 = 0; i0 < NIT; i0 += BATCH) {
                        uint4 code[BATCH];
#pragma unroll
                        for (int u = 0; u < BATCH; ++u) {
                            const int j = keys[r8 + (i0 + u) * RPI8];
                            code[u] = j >= 0 ? ld_codes16(src0 + (int64_t)j * row_bytes) : make_uint4(0u, 0u, 0u, 0u);
                        }
#pragma unroll
                        for (int u = 0; u < BATCH; ++u) {
                            const int r = r8 + (i0 + u) * RPI8;
                            const uint32_t w[4] = {code[u].x, code[u].y, code[u].z, code[u].w};
                            uint32_t o[8];
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4) {
                                o[2 * k4] = e4m3x2_to_bf16x2(w[k4]);
                                o[2 * k4 + 1] = e4m3x2_to_bf16x2(w[k4] >> 16);
                            }
                            const uint32_t row_dst = dst8 + r * 128;
                            const int cb = (2 * c8) & 7;   // chunk inside the 64-dim slice: cb and cb + 1
                            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(row_dst + ((cb ^ (r & 7)) << 4)), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
                            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(row_dst + (((cb + 1) ^ (r & 7)) << 4)), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7]) : "memory");
                        }
                    }
                    mbar_arrive(bar(bar_full + st));   // (release: this thread's stores are visible to whoever observes the phase)
                }
            }
        }
        cp_async_wait_all();   // nothing of this thread stays in flight, also on the abort path
        if (!is_v && gtid == 0 && *abort_flag)
            for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar(Q_FULL), (n - 1) & 1); ++it) {}
    }
    // ------------------------------------------------ cluster merge (every thread of every CTA of the cluster comes here,
    // whatever happened before: a CTA that gave up still arrives, its partial is then not valid and the error word says so)
    if (n_splits > 1 && part_o == nullptr) {
        __syncwarp();
        cluster_sync_all();   // all partials are parked
        if (is_softmax_warp(warp) && (int64_t)blockIdx.x < n_items) {
            uint32_t my_rank;
            asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(my_rank));
            const Where q = where(blockIdx.x);
            const int quad = warp & 1, half = warp >> 2;
            const int row = 32 * quad + lane;
            const bool real = row < min(kSubHeads, p.G - kSubHeads * q.sub);
            const int h = q.gkv * p.G + kSubHeads * q.sub + (real ? row : 0);
            const int W = D / n_splits, Wt = W / 2;            // this CTA's column slice, this thread's half of it
            const int col0 = (int)my_rank * W + half * Wt;
            float m = -INFINITY;
            for (int r = 0; r < n_splits; ++r)
                m = fmaxf(m, ld_peer2(peer_smem(sbase + C::kOffPartMl + row * 8, r)).x);
            float l = 0.f;
            float4 acc[D / 16];                                // Wt / 4 <= D / 16 entries are used
#pragma unroll
            for (int u = 0; u < D / 16; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int r = 0; r < n_splits; ++r) {
                const float2 ml = ld_peer2(peer_smem(sbase + C::kOffPartMl + row * 8, r));
                const float f = ml.x == -INFINITY ? 0.f : exp2f(ml.x - m);
                l += f * ml.y;
                const uint32_t src = peer_smem(sbase + C::kOffK + row * C::kPartPitch + col0 * 4, r);
#pragma unroll
                for (int u = 0; u < D / 16; ++u)
                    if (4 * u < Wt) {
                        const float4 v = ld_peer4(src + u * 16);
                        acc[u].x += f * v.x; acc[u].y += f * v.y; acc[u].z += f * v.z; acc[u].w += f * v.w;
                    }
            }
            if (real) {
                const float inv = l > 0.f ? 1.f / l : 0.f;
                const int64_t o_off = q.b * p.os_b + (int64_t)q.i * p.os_t + h * p.os_h + col0;
#pragma unroll
                for (int u = 0; u < D / 16; ++u)
                    if (4 * u < Wt) {
                        if (p.gate) {
                            const uint2 gv = *reinterpret_cast<const uint2 *>(static_cast<const __nv_bfloat16 *>(p.gate) + o_off + u * 4);
                            const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gv.x));
                            const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gv.y));
                            acc[u].x *= gate_of(g0.x); acc[u].y *= gate_of(g0.y); acc[u].z *= gate_of(g1.x); acc[u].w *= gate_of(g1.y);
                        }
                        uint2 v;
                        v.x = pack_bf16(acc[u].x * inv, acc[u].y * inv);
                        v.y = pack_bf16(acc[u].z * inv, acc[u].w * inv);
                        *reinterpret_cast<uint2 *>(O + o_off + u * 4) = v;
                    }
                if (my_rank == 0 && half == 0 && LSE) LSE[((int64_t)q.b * p.Hq + h) * p.Lq + q.i] = l > 0.f ? (m + log2f(l)) * kLn2 : -INFINITY;
            }
        }
        __syncwarp();
        cluster_sync_all();   // nobody leaves (and frees its shared memory) while a peer still reads it
    }
    // ------------------------------------------------ teardown
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(C::kTmem) : "memory");
    }
}

constexpr int kMaxSplits = 16;

// Combines the n_splits partials of every (query, head): one warp per pair.  Lane sp fetches the (maximum, sum) of
// split sp, so all of them are in flight at once; the accumulator rows are then read with independent loads.
template <int D>
__global__ void __launch_bounds__(256)
k_sparse_tc5_combine(const Params p, const float *__restrict__ part_ml, const float *__restrict__ part_o,
                     __nv_bfloat16 *__restrict__ O, float *__restrict__ LSE, int n_sub, int n_splits, int64_t n_pairs)
{
    const int lane = threadIdx.x & 31;
    const int64_t pair = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // (b, i, head)
    if (pair >= n_pairs) return;
    const int h = (int)(pair % p.Hq);
    const int64_t bi = pair / p.Hq;
    const int i = (int)(bi % p.Lq), b = (int)(bi / p.Lq);
    const int gkv = h / p.G, hh = h % p.G;
    const int sub = hh / kSubHeads, row = hh % kSubHeads;
    const int64_t item0 = ((((int64_t)b * p.Hkv + gkv) * n_sub + sub) * p.Lq + i) * n_splits;
    float2 ml = make_float2(-INFINITY, 0.f);
    if (lane < n_splits) ml = *reinterpret_cast<const float2 *>(part_ml + ((item0 + lane) * kSubHeads + row) * 2);
    const float m = warp_max(ml.x);
    const float f_mine = ml.x == -INFINITY ? 0.f : exp2f(ml.x - m);
    const float l = warp_sum(f_mine * ml.y);
    constexpr int NV = D / 128;   // float4 per lane
    float4 acc[NV];
#pragma unroll
    for (int u = 0; u < NV; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    const float *po = part_o + (item0 * kSubHeads + row) * D + lane * 4;
#pragma unroll 4
    for (int sp = 0; sp < n_splits; ++sp) {
        const float f = __shfl_sync(0xffffffffu, f_mine, sp);
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const float4 v = *reinterpret_cast<const float4 *>(po + (int64_t)sp * kSubHeads * D + u * 128);
            acc[u].x += f * v.x; acc[u].y += f * v.y; acc[u].z += f * v.z; acc[u].w += f * v.w;
        }
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const int64_t o_off = b * p.os_b + (int64_t)i * p.os_t + h * p.os_h + lane * 4;
    __nv_bfloat16 *orow = O + o_off;
#pragma unroll
    for (int u = 0; u < NV; ++u) {
        if (p.gate) {
            const uint2 gv = *reinterpret_cast<const uint2 *>(static_cast<const __nv_bfloat16 *>(p.gate) + o_off + u * 128);
            const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gv.x));
            const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gv.y));
            acc[u].x *= gate_of(g0.x); acc[u].y *= gate_of(g0.y); acc[u].z *= gate_of(g1.x); acc[u].w *= gate_of(g1.y);
        }
        uint2 v;
        v.x = pack_bf16(acc[u].x * inv, acc[u].y * inv);
        v.y = pack_bf16(acc[u].z * inv, acc[u].w * inv);
        *reinterpret_cast<uint2 *>(orow + u * 128) = v;
    }
    if (lane == 0 && LSE) LSE[((int64_t)b * p.Hq + h) * p.Lq + i] = l > 0.f ? (m + log2f(l)) * kLn2 : -INFINITY;
}

constexpr int kPlanSms = 148;   // the workspace is sized for this many SMs; a launch on another part adapts to what it got

struct SplitPlan { int n_sub, n_splits, nblk; int64_t queries; };

// Splits over the keys only when the queries alone cannot fill the SMs (decode, very short prefill chunks).
SplitPlan plan_splits(const Params &p, int n_sm, bool allow_split)
{
    SplitPlan pl;
    pl.n_sub = (p.G + kSubHeads - 1) / kSubHeads;
    pl.queries = (int64_t)p.B * p.Hkv * pl.n_sub * p.Lq;
    const int tiles = (p.k + p.w + BN - 1) / BN;
    int ns = 1;
    if (allow_split && pl.queries > 0 && pl.queries < n_sm) {
        ns = (int)(n_sm / pl.queries);
        if (ns > kMaxSplits) ns = kMaxSplits;
        if (ns > tiles) ns = tiles;
        if (ns < 1) ns = 1;
    }
    pl.nblk = (tiles + ns - 1) / ns;
    pl.n_splits = (tiles + pl.nblk - 1) / pl.nblk;   // no run of tiles is entirely past the slot array
    return pl;
}
size_t split_ws_bytes(const Params &p, const SplitPlan &pl)
{
    if (pl.n_splits <= 1) return 0;
    return (size_t)pl.queries * pl.n_splits * kSubHeads * (p.D + 2) * sizeof(float);
}

template <int D, bool F8>
cudaError_t launch_sp(const Params &p, const void *Q, const void *K, const void *V, const float *ksc, const float *vsc,
                      const int32_t *idx, const float *sink, void *O, float *LSE, void *ws, size_t ws_bytes, bool allow_split,
                      cudaStream_t st)
{
    using C = SpCfg<D, F8>;
    CUtensorMap tmQ;
    const int box_heads = p.G < kSubHeads ? p.G : kSubHeads;
    if (!make_tile_map(&tmQ, Q, p.B, p.Lq, p.Hq, p.qs_b, p.qs_t, p.qs_h, 1, box_heads, D)) return cudaErrorNotSupported;
    static bool attr_set[64] = {};
    static int n_sm[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorNotSupported;
    if (!attr_set[dev]) {
        if ((e = cudaFuncSetAttribute(k_sparse_tc5<D, F8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kSmemBytes)) != cudaSuccess) return e;
        if ((e = cudaDeviceGetAttribute(&n_sm[dev], cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    // Few queries: the keys of a query are split over CTAs.  The splits of a query are a thread-block cluster that merges
    // through distributed shared memory (no scratch, one launch) when their number can be a power of two up to 8;
    // otherwise, with scratch, partials go through global memory and a second kernel combines them.
    SplitPlan pl = plan_splits(p, n_sm[dev] * C::kMinBlocks, allow_split && (ws != nullptr || HS2_SPTC5_CLUSTER));
    bool by_cluster = false;
    if (HS2_SPTC5_CLUSTER && pl.n_splits > 1) {
        const int tiles = (p.k + p.w + BN - 1) / BN;
        int c = 8;
        while (c > pl.n_splits) c >>= 1;          // largest power of two within the planned split and the cluster limit
        pl.nblk = (tiles + c - 1) / c;            // (runs past the slot array are void and merge as nothing)
        pl.n_splits = c;
        by_cluster = true;
    } else if (split_ws_bytes(p, pl) > ws_bytes) {
        pl = plan_splits(p, 1, false);            // scratch too small for this part: no split
    }
    const int64_t items = pl.queries * pl.n_splits;
    if (items <= 0) return cudaSuccess;
    float *part_ml = by_cluster ? nullptr : reinterpret_cast<float *>(ws);
    float *part_o = (pl.n_splits > 1 && !by_cluster) ? part_ml + items * kSubHeads * 2 : nullptr;
    const int64_t resident = (int64_t)n_sm[dev] * C::kMinBlocks;
    const unsigned grid = (unsigned)(by_cluster ? items : (items < resident ? items : resident));
    if (by_cluster) {
        if (items > 0x7fffffffLL) return cudaErrorNotSupported;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(C::kThreads);
        cfg.dynamicSmemBytes = C::kSmemBytes;
        cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = (unsigned)pl.n_splits;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, k_sparse_tc5<D, F8>, tmQ, p, K, V, ksc, vsc, idx, sink, (__nv_bfloat16 *)O, LSE, items, pl.n_sub,
                               pl.n_splits, pl.nblk, (float *)nullptr, (float *)nullptr);
        count_launch();
        return e != cudaSuccess ? e : cudaGetLastError();
    }
    k_sparse_tc5<D, F8><<<grid, C::kThreads, C::kSmemBytes, st>>>(
        tmQ, p, K, V, ksc, vsc, idx, sink, (__nv_bfloat16 *)O, LSE, items, pl.n_sub, pl.n_splits, pl.nblk, part_ml, part_o);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess || pl.n_splits <= 1) return e;
    const int64_t n_pairs = (int64_t)p.B * p.Lq * p.Hq;
    // (a programmatic dependent launch of this kernel was measured: 23 -> 31 us per decode step at batch 16, so it is
    // launched the plain way)
    k_sparse_tc5_combine<D><<<(unsigned)((n_pairs + 7) / 8), 256, 0, st>>>(p, part_ml, part_o, (__nv_bfloat16 *)O, LSE, pl.n_sub,
                                                                       pl.n_splits, n_pairs);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

// bf16; head_dim 256 with up to 128 query heads per KV head, head_dim 128 with 9 to 128
bool sparse_tc5_supported_shape(const Params &p, hs2_dtype dt)
{
    auto m8 = [](int64_t x) { return x % 8 == 0 && x > 0; };
    if (p.ks_t * 2 > 0x7fffffffLL) return false;
    // at head_dim 128 groups of up to 8 belong to the mma.sync gather kernel; at 256 this is the only tensor-core one
    return dt == HS2_BF16 && (p.D == 256 || (p.D == 128 && p.G > 8)) && p.G >= 1 && p.G <= 128 && m8(p.qs_b) && m8(p.qs_t) && m8(p.qs_h) &&
           m8(p.ks_b) && m8(p.ks_t) && m8(p.ks_h) && m8(p.os_b) && m8(p.os_t) && m8(p.os_h) &&
           (int64_t)p.B * p.Hkv * p.Lq * 2 * kMaxSplits <= 0x7fffffffLL && p.k + p.w > 0;
}
bool sparse_tc5_supported(const Params &p, hs2_dtype dt) { return sparse_tc5_supported_shape(p, dt) && tma_available(); }

// Scratch for splitting the keys of a query over several CTAs (sized for a 148-SM part; 0 when no split pays).
size_t sparse_tc5_ws_bytes(const Params &p)
{
    return split_ws_bytes(p, plan_splits(p, kPlanSms * (p.D <= 128 ? 2 : 1), true));
}

// Returns cudaErrorNotSupported when the tensor map cannot be built (the caller then takes the generic kernel).
// ws may be null: the keys of a query are then never split.
cudaError_t launch_sparse_tc5(const Params &p, const void *Q, const void *K, const void *V, const int32_t *idx,
                              const float *sink, void *O, float *LSE, void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (p.D == 128) return launch_sp<128, false>(p, Q, K, V, nullptr, nullptr, idx, sink, O, LSE, ws, ws_bytes, true, st);
    if (p.D == 256) return launch_sp<256, false>(p, Q, K, V, nullptr, nullptr, idx, sink, O, LSE, ws, ws_bytes, true, st);
    return cudaErrorNotSupported;
}

// The same on an e4m3 cache (codes + one fp32 scale per (token, KV head)); bf16 queries and outputs.  The strides of
// `p` for K and V count codes.  ws as above (null: the keys of a query are never split).
bool sparse_tc5_fp8_supported(const Params &p, hs2_dtype dt)
{
    auto m8 = [](int64_t x) { return x % 8 == 0 && x > 0; };
    auto m16 = [](int64_t x) { return x % 16 == 0 && x > 0; };
    if (p.ks_t > 0x7fffffffLL) return false;
    return dt == HS2_BF16 && (p.D == 256 || p.D == 128) && p.G >= 1 && p.G <= 128 && m8(p.qs_b) && m8(p.qs_t) && m8(p.qs_h) &&
           m16(p.ks_b) && m16(p.ks_t) && m16(p.ks_h) && m8(p.os_b) && m8(p.os_t) && m8(p.os_h) &&
           (int64_t)p.B * p.Hkv * p.Lq * 2 * kMaxSplits <= 0x7fffffffLL && p.k + p.w > 0 && tma_available();
}
cudaError_t launch_sparse_tc5_fp8(const Params &p, const void *Q, const void *K8, const void *V8, const float *ksc,
                                  const float *vsc, const int32_t *idx, const float *sink, void *O, float *LSE, void *ws,
                                  size_t ws_bytes, cudaStream_t st)
{
    if (p.D == 128) return launch_sp<128, true>(p, Q, K8, V8, ksc, vsc, idx, sink, O, LSE, ws, ws_bytes, true, st);
    if (p.D == 256) return launch_sp<256, true>(p, Q, K8, V8, ksc, vsc, idx, sink, O, LSE, ws, ws_bytes, true, st);
    return cudaErrorNotSupported;
}

cudaError_t read_sparse_tc5_error(unsigned *out)
{
    return cudaMemcpyFromSymbol(out, g_sptc5_error, sizeof(unsigned));
}

}  // namespace hs2
