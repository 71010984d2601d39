// Sparse attention over (reused top-k indices) U (forced window) for bf16, head_dim 128, group <= 8
// (Section 3.3: both selected sets are read from the full-attention layer's KV cache).
//
// The work is a gather: per (query, KV head) up to k+w rows of K and of V, 256 bytes each, are
// fetched once and shared by the G query heads of the group.  It is bound by memory, so the design
// goal is bytes in flight, not flops:
//   * one warp owns one (query, KV head) item (prefill) or one split of it (decode) and runs its own
//     cp.async pipeline: NSTAGE stages of KT key rows (K and V), 16-byte copies, rows placed in
//     shared memory with an XOR swizzle so that ldmatrix is conflict free; no CTA-wide barriers.
//     Prefill (cache mostly in L2) runs with ONE buffer per warp - fetch, wait, fold: the latency of a
//     warp's fetch is covered by the other warps.  Measured on the 8K benchmark: two stages of 16 rows x
//     12 warps 1.47 ms; one buffer of 16 rows x 20 warps 1.23 ms; one buffer of 32 rows x 12 warps
//     1.19 ms (the default).  Decode (cache in HBM, few tiles per warp) keeps two stages of 16 rows;
//   * the G x keys products go through tensor cores only because plain FMAs could not keep up with
//     the memory system at 8 flop/byte: S^T = K Q^T with the keys on the MMA M dimension and the
//     (padded to 8) heads on N, so nothing of the m16n8k16 tile is wasted; P^T is re-laid out for the
//     second product with movmatrix; O^T = V^T P^T reads V through ldmatrix.trans;
//   * online softmax in the base-2 domain with warp shuffles across the 8 key rows of a fragment.
// Decode splits the attended set of one (sequence, KV head) over several warps; each writes an
// un-normalised partial (m, l, O) and the last one to arrive (an atomic ticket, nobody waits) merges.
#include <atomic>
#include <mutex>

#include "hs2_common.cuh"

// Tuning knobs (compile time): key rows per stage, pipeline depth, warps per CTA; prefill and decode.
#ifndef HS2_SP_KT
#define HS2_SP_KT 32
#endif
#ifndef HS2_SP_NSTAGE
#define HS2_SP_NSTAGE 1
#endif
#ifndef HS2_SP_WARPS
#define HS2_SP_WARPS 12
#endif
#ifndef HS2_SPD_KT
#define HS2_SPD_KT 16
#endif
#ifndef HS2_SPD_NSTAGE
#define HS2_SPD_NSTAGE 2
#endif
#ifndef HS2_SPD_WARPS
#define HS2_SPD_WARPS 6
#endif
// 1: rows are fetched with one bulk async copy (TMA, 256 bytes) per row that completes on an mbarrier;
// 0: sixteen 16-byte cp.async per row.
#ifndef HS2_SP_BULK
#define HS2_SP_BULK 0
#endif
// 1: the prefill kernel fetches the K rows and the V rows of a tile as separate copy groups and overlaps each with the
// other half's arithmetic inside the warp; 0: one fetch, one wait, one fold per tile.
#ifndef HS2_SP_OVERLAP
#define HS2_SP_OVERLAP 0
#endif

namespace hs2 {
namespace {

constexpr int HD = 128;                      // head_dim
constexpr int kRowBytes = HD * 2;            // one K or V row
constexpr bool kBulk = HS2_SP_BULK != 0;
// row pitch in shared memory: bulk copies cannot swizzle, so rows are padded by 16 bytes instead
// (17 sixteen-byte units per row: eight consecutive rows hit eight different bank groups)
constexpr int kPitch = kBulk ? kRowBytes + 16 : kRowBytes;
__device__ unsigned g_sparse_error;          // bit 0: a bounded mbarrier wait ran out
constexpr int kMaxSplits = 32;               // warp-level splits of one (sequence, KV head) in decode

// KT key rows per pipeline stage (16 or 32), NSTAGE stages per warp, WARPS warps per CTA
template <int KT_, int NSTAGE_, int WARPS_>
struct Cfg {
    static constexpr int KT = KT_, NSTAGE = NSTAGE_, WARPS = WARPS_;
    static constexpr int kStageBytes = 2 * KT * kPitch;                          // K tile then V tile
    static constexpr int kWarpSmem = NSTAGE * kStageBytes + NSTAGE * 32 * 4 + 64;   // + key index of each staged row + mbarriers
    static_assert(KT == 16 || KT == 32, "a stage holds 16 or 32 key rows");
    static_assert(NSTAGE >= 1, "at least one buffer");
};
using PrefillCfg = Cfg<HS2_SP_KT, HS2_SP_NSTAGE, HS2_SP_WARPS>;
using DecodeCfg = Cfg<HS2_SPD_KT, HS2_SPD_NSTAGE, HS2_SPD_WARPS>;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes)
{
    // (.cg: past L1.  Copies that allocate in L1, .ca, were measured: 1.47 vs 1.14 ms per layer at 8K, 23.1 vs 17.6 ms at
    // 2 x 32K - what is left of L1 beside 197 KB of shared memory is too small for the rows neighbouring queries share)
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_copy_row(uint32_t dst, const void *src, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], 256, [%2];\n"
                 ::"r"(dst), "l"(src), "r"(bar) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Accumulators of one warp.  Thread (g = lane/4, t = lane%4) owns heads 2t and 2t+1 of the group:
// o[dt][0..3] = O^T at (d = 16 dt + g, head 2t), (same d, head 2t+1), (d + 8, head 2t), (d + 8, head 2t+1);
// m is replicated over g, l is this thread's partial sum (reduced over g at the end).
struct Acc {
    float o[8][4];
    float m[2], l[2];
};

struct Item {
    const char *Kb, *Vb;      // first row of this (sequence, KV head), bytes
    int64_t row_stride;       // bytes between consecutive tokens
    const int32_t *irow;      // idx row of this (query, KV head), or nullptr when k == 0
    int pos, kvl;
    float *raw;               // optional: raw q.k of every (head, key) of this pair, [G][lk] (decode-shaped full layer)
    int lk;
};

// Slot s of the virtual slot array [idx row | window] holds a key index or is void (-1).  slot_raw starts the fetch
// (an idx entry is a global load), slot_fix applies the validity rules when the value is used one tile later, so
// that the load's latency is never waited for.
template <int KT>
__device__ __forceinline__ int slot_raw(const Params &p, const Item &it, int tile, int lane)
{
    const int s = tile * KT + lane;
    if (lane >= KT) return -1;
    if (s < p.k) return __ldg(it.irow + s);
    return s < p.k + p.w ? it.pos - p.w + 1 + (s - p.k) : -1;
}
template <int KT>
__device__ __forceinline__ int slot_fix(const Params &p, const Item &it, int tile, int lane, int j)
{
    const int hi = tile * KT + lane < p.k ? it.pos - p.w : it.pos;   // idx entries inside the window are void
    return (j < 0 || j > hi || j >= it.kvl) ? -1 : j;
}

// bulk variant: lane r < KT copies K row r, lane 16 + r copies V row r; void rows are not copied (the stage
// buffers start zeroed and only ever receive real rows, so stale rows are finite and get probability 0)
template <int KT>
__device__ __forceinline__ void issue_stage_bulk(const Item &it, uint32_t stage_base, uint32_t bar, int j, int lane)
{
    static_assert(KT == 16, "the bulk variant maps one K and one V row to each lane");
    const int r = lane & 15, hi = lane >> 4;
    const int jr = __shfl_sync(0xffffffffu, j, r);
    const unsigned valid = __ballot_sync(0xffffffffu, jr >= 0) & 0xffffu;
    if (lane == 0) mbar_expect_tx(bar, __popc(valid) * 2u * kRowBytes);
    __syncwarp();
    if (jr >= 0) {
        const char *src = (hi ? it.Vb : it.Kb) + (int64_t)jr * it.row_stride;
        bulk_copy_row(stage_base + hi * KT * kPitch + r * kPitch, src, bar);
    }
}

template <int KT>
__device__ __forceinline__ void issue_stage(const Item &it, uint32_t stage_base, int j, int lane)
{
    // lane -> 16-byte chunk c of rows r0 + (lane >> 4), r0 = 0, 2, 4, ...  Because r0 is even,
    // (c ^ (r & 7)) = (c ^ (lane >> 4)) ^ (r0 & 6): the lane part is hoisted, the rest is a constant.
    const int c = lane & 15, hi = lane >> 4;
    const uint32_t cx = (uint32_t)(c ^ hi);
    const uint32_t dst_lane = stage_base + hi * kRowBytes;
    const char *kc = it.Kb + c * 16, *vc = it.Vb + c * 16;
    const int rs = (int)it.row_stride;
#pragma unroll
    for (int r0 = 0; r0 < KT; r0 += 2) {
        const int jr = __shfl_sync(0xffffffffu, j, r0 + hi);
        const uint32_t dst = dst_lane + r0 * kRowBytes + ((cx ^ (uint32_t)(r0 & 6)) << 4);
        const int64_t off = (int64_t)max(jr, 0) * rs;   // one wide multiply-add per tensor
        const int nbytes = jr < 0 ? 0 : 16;             // void rows are zero filled, nothing is read
        cp_async16(dst, kc + off, nbytes);
        cp_async16(dst + KT * kRowBytes, vc + off, nbytes);
    }
}

// one tensor's rows of a tile (K into the first half of a stage, V into the second): the overlapped prefill loop
// fetches the two halves at different times
template <int KT>
__device__ __forceinline__ void issue_rows(const char *tensor_base, int rs, uint32_t dst_base, int j, int lane)
{
    const int c = lane & 15, hi = lane >> 4;
    const uint32_t cx = (uint32_t)(c ^ hi);
    const uint32_t dst_lane = dst_base + hi * kRowBytes;
    const char *tc = tensor_base + c * 16;
#pragma unroll
    for (int r0 = 0; r0 < KT; r0 += 2) {
        const int jr = __shfl_sync(0xffffffffu, j, r0 + hi);
        const uint32_t dst = dst_lane + r0 * kRowBytes + ((cx ^ (uint32_t)(r0 & 6)) << 4);
        cp_async16(dst, tc + (int64_t)max(jr, 0) * rs, jr < 0 ? 0 : 16);   // void rows are zero filled, nothing is read
    }
}

// S^T = K Q^T of one stage: rows = keys, columns = heads.  Two accumulator chains per tile keep the tensor pipe busy.
template <int KT>
__device__ __forceinline__ void stage_scores(float (&s)[KT / 16][4], const uint32_t (&qf)[16], uint32_t stage_base, int lane)
{
    const int mi = lane >> 3, rr = lane & 7;
    constexpr int MT = KT / 16;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        float s2[4] = {0.f, 0.f, 0.f, 0.f};
        s[mt][0] = s[mt][1] = s[mt][2] = s[mt][3] = 0.f;
        // chunk = 2 ks + (mi >> 1); (chunk ^ rr) << 4 = (32 ks) ^ lx with lx = ((mi >> 1) ^ rr) << 4
        const uint32_t rowaddr = stage_base + (mt * 16 + (mi & 1) * 8 + rr) * kPitch;
        const uint32_t lx = kBulk ? (uint32_t)(mi >> 1) << 4 : (uint32_t)((mi >> 1) ^ rr) << 4;   // padded rows need no swizzle
#pragma unroll
        for (int ks = 0; ks < 8; ks += 2) {
            uint32_t a[4], a2[4];
            ldmatrix_x4(a, rowaddr + (kBulk ? lx + (uint32_t)(32 * ks) : lx ^ (uint32_t)(32 * ks)));
            ldmatrix_x4(a2, rowaddr + (kBulk ? lx + (uint32_t)(32 * ks + 32) : lx ^ (uint32_t)(32 * ks + 32)));
            mma_bf16(s[mt], a, qf[2 * ks], qf[2 * ks + 1]);
            mma_bf16(s2, a2, qf[2 * ks + 2], qf[2 * ks + 3]);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) s[mt][e] += s2[e];
    }
}

// online softmax of one stage in the base-2 domain; this thread: heads 2t+hh, keys 16 mt + g + 8 r.  Leaves the
// probabilities as the bf16 B operand of the second product and rescales the accumulator when a maximum moved.
template <int KT>
__device__ __forceinline__ void stage_softmax(Acc &acc, float (&s)[KT / 16][4], uint32_t (&pb)[KT / 16][2], unsigned mask,
                                              float scale_log2, int lane)
{
    const int g = lane >> 2;
    constexpr int MT = KT / 16;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const bool ok = (mask >> (mt * 16 + g + 8 * r)) & 1u;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const float t2 = ok ? s[mt][2 * r + hh] * scale_log2 : -INFINITY;
                s[mt][2 * r + hh] = t2;
                mx[hh] = fmaxf(mx[hh], t2);
            }
        }
    float corr[2], muse[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 4));
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 8));
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 16));
        const float m_new = fmaxf(acc.m[hh], mx[hh]);
        muse[hh] = m_new == -INFINITY ? 0.f : m_new;
        corr[hh] = exp2f(acc.m[hh] - muse[hh]);
        acc.m[hh] = m_new;
        acc.l[hh] *= corr[hh];
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        float pv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            pv[e] = exp2f(s[mt][e] - muse[e & 1]);
            acc.l[e & 1] += pv[e];
        }
        pb[mt][0] = movmatrix_trans(pack_bf16(pv[0], pv[1]));   // keys 16 mt + 0..7
        pb[mt][1] = movmatrix_trans(pack_bf16(pv[2], pv[3]));   // keys 16 mt + 8..15
    }
    if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {   // the running max moved for some head
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
            acc.o[dt][0] *= corr[0]; acc.o[dt][1] *= corr[1];
            acc.o[dt][2] *= corr[0]; acc.o[dt][3] *= corr[1];
        }
    }
}

// O^T += V^T P^T : rows = output dimensions, contraction over the keys of the stage (vbase: the stage's V rows)
template <int KT>
__device__ __forceinline__ void stage_pv(Acc &acc, const uint32_t (&pb)[KT / 16][2], uint32_t vbase, int lane)
{
    const int mi = lane >> 3, rr = lane & 7;
    constexpr int MT = KT / 16;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const uint32_t rowaddr = vbase + (mt * 16 + (mi >> 1) * 8 + rr) * kPitch;
        const uint32_t lx = kBulk ? (uint32_t)(mi & 1) << 4 : (uint32_t)((mi & 1) ^ rr) << 4;
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
            uint32_t a[4];
            ldmatrix_x4_trans(a, rowaddr + (kBulk ? lx + (uint32_t)(32 * dt) : lx ^ (uint32_t)(32 * dt)));
            mma_bf16(acc.o[dt], a, pb[mt][0], pb[mt][1]);
        }
    }
}

template <int KT>
__device__ __forceinline__ void consume_stage(Acc &acc, const uint32_t (&qf)[16], uint32_t stage_base, unsigned mask,
                                              float scale_log2, int lane, float *raw = nullptr, int lk = 0, int G = 0,
                                              const int *sjrow = nullptr)
{
    constexpr int MT = KT / 16;
    float s[MT][4];
    stage_scores<KT>(s, qf, stage_base, lane);
    if (raw) {
        // The decode-shaped full layer keeps the raw products: the selection scores need the final LSE, and reading
        // them back (4 bytes per head and key) is far cheaper than sweeping K a second time.
        const int g = lane >> 2, t = lane & 3;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int j = sjrow[mt * 16 + g + 8 * r];
                if (j >= 0) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh)
                        if (2 * t + hh < G) raw[(int64_t)(2 * t + hh) * lk + j] = s[mt][2 * r + hh];
                }
            }
    }
    uint32_t pb[MT][2];
    stage_softmax<KT>(acc, s, pb, mask, scale_log2, lane);
    stage_pv<KT>(acc, pb, stage_base + KT * kPitch, lane);
}

// Fold slot tiles [t_begin, t_end) of one item into acc with an NSTAGE-deep cp.async pipeline.
template <class C>
__device__ __forceinline__ void run_tiles(const Params &p, const Item &it, const uint32_t (&qf)[16], Acc &acc,
                                          int t_begin, int t_end, char *wsm, int lane)
{
    constexpr int KT = C::KT, NSTAGE = C::NSTAGE, kStageBytes = C::kStageBytes;
    const uint32_t sbase = smem_u32(wsm);
    int *sj = reinterpret_cast<int *>(wsm + NSTAGE * kStageBytes);
    const uint32_t bars = sbase + NSTAGE * kStageBytes + NSTAGE * 32 * 4;   // one mbarrier per stage (bulk variant)
    if (kBulk) {
        // zero the stage buffers once (void rows are never copied), set up the barriers
        uint4 *z = reinterpret_cast<uint4 *>(wsm);
        for (int e = lane; e < NSTAGE * kStageBytes / 16; e += 32) z[e] = make_uint4(0u, 0u, 0u, 0u);
        if (lane == 0)
            for (int s2 = 0; s2 < NSTAGE; ++s2) mbar_init(bars + 8 * s2, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
        __syncwarp();
    }
    int next = t_begin;
    int jn = next < t_end ? slot_raw<KT>(p, it, next, lane) : -1;
    int n_issued = 0, n_done = 0;
    auto try_issue = [&](int stage) -> bool {
        while (next < t_end) {
            const int j = slot_fix<KT>(p, it, next, lane, jn);
            ++next;
            if (next < t_end) jn = slot_raw<KT>(p, it, next, lane);
            if (__ballot_sync(0xffffffffu, j >= 0)) {
                sj[stage * 32 + lane] = j;
                if constexpr (kBulk) issue_stage_bulk<KT>(it, sbase + stage * kStageBytes, bars + 8 * stage, j, lane);
                else issue_stage<KT>(it, sbase + stage * kStageBytes, j, lane);
                return true;
            }
        }
        return false;
    };
    if (HS2_SP_OVERLAP && NSTAGE == 1 && !kBulk && !it.raw) {
        // Built and measured, not the default (HS2_SP_OVERLAP=1): 72.5 vs 68.5 ms per layer at 128K, 18.7 vs 17.6 ms at
        // 2 x 32K, 1.18 vs 1.14 ms at 8K.  The other warps of the SM already cover a warp's fetch; two waits and half-sized
        // copy bursts per tile cost more than the overlap inside one warp returns.
        // One buffer per warp, its K half and its V half fetched at different times so that most of each fetch hides
        // behind the other half's arithmetic:
        //   V(t) is issued, K(t) awaited, S = K Q^T; K(t+1) is issued into the K half just read; softmax;
        //   V(t) awaited, O += P V.  Two copy groups are in flight at any time and each wait leaves the younger one.
        constexpr int MT = KT / 16;
        const int rs = (int)it.row_stride;
        auto next_tile = [&](int &j) -> bool {   // the next tile with a live slot
            while (next < t_end) {
                j = slot_fix<KT>(p, it, next, lane, jn);
                ++next;
                if (next < t_end) jn = slot_raw<KT>(p, it, next, lane);
                if (__ballot_sync(0xffffffffu, j >= 0)) return true;
            }
            return false;
        };
        int jc;
        if (!next_tile(jc)) return;
        issue_rows<KT>(it.Kb, rs, sbase, jc, lane);
        cp_async_commit();
        while (true) {
            issue_rows<KT>(it.Vb, rs, sbase + KT * kRowBytes, jc, lane);
            cp_async_commit();
            const unsigned mask = __ballot_sync(0xffffffffu, jc >= 0);
            cp_async_wait<1>();   // K(t) has landed; V(t) may still be on its way
            __syncwarp();
            float s[MT][4];
            stage_scores<KT>(s, qf, sbase, lane);
            __syncwarp();         // every lane has read the K half before the next tile's rows land in it
            int jnext = -1;
            const bool more = next_tile(jnext);
            if (more) issue_rows<KT>(it.Kb, rs, sbase, jnext, lane);
            cp_async_commit();    // (an empty group after the last tile keeps the counting uniform)
            uint32_t pb[MT][2];
            stage_softmax<KT>(acc, s, pb, mask, p.scale_log2, lane);
            cp_async_wait<1>();   // V(t) has landed; K(t+1) may still be on its way
            __syncwarp();
            stage_pv<KT>(acc, pb, sbase + KT * kRowBytes, lane);
            __syncwarp();         // every lane has read the V half before the next tile's rows land in it
            if (!more) break;
            jc = jnext;
        }
        cp_async_wait<0>();
        return;
    }
    if (NSTAGE == 1 && !kBulk) {
        // one buffer per warp: fetch, wait, fold (the variant that also keeps the raw products)
        while (try_issue(0)) {
            cp_async_commit();
            cp_async_wait<0>();
            __syncwarp();
            const unsigned mask = __ballot_sync(0xffffffffu, sj[lane] >= 0);
            consume_stage<KT>(acc, qf, sbase, mask, p.scale_log2, lane, it.raw, it.lk, p.G, sj);
            __syncwarp();   // every lane has read the buffer before the next tile's copies land in it
        }
        return;
    }
#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (try_issue(n_issued % NSTAGE)) ++n_issued;
        if (!kBulk) cp_async_commit();
    }
    bool gave_up = false;
    while (n_done < n_issued) {
        const int stage = n_done % NSTAGE;
        if (kBulk) {
            // bounded wait for the stage's rows; the parity of a stage flips every NSTAGE tiles
            const uint32_t parity = (uint32_t)(n_done / NSTAGE) & 1u;
            bool ok = false;
            for (uint32_t spin = 0; spin < (1u << 22) && !ok; ++spin) ok = mbar_try_wait(bars + 8 * stage, parity);
            if (!__all_sync(0xffffffffu, ok)) {
                if (lane == 0) atomicOr(&g_sparse_error, 1u);
                gave_up = true;
                break;
            }
        } else {
            cp_async_wait<(NSTAGE >= 2 ? NSTAGE - 2 : 0)>();
        }
        __syncwarp();
        if (try_issue(n_issued % NSTAGE)) ++n_issued;
        if (!kBulk) cp_async_commit();
        const unsigned mask = __ballot_sync(0xffffffffu, sj[stage * 32 + lane] >= 0);
        consume_stage<KT>(acc, qf, sbase + stage * kStageBytes, mask, p.scale_log2, lane, it.raw, it.lk, p.G, sj + stage * 32);
        ++n_done;
    }
    if (kBulk) {
        if (gave_up) {   // let the copies that are still in flight land before the buffers are reused
            for (int t = n_done; t < n_issued; ++t) {
                const uint32_t parity = (uint32_t)(t / NSTAGE) & 1u;
                for (uint32_t spin = 0; spin < (1u << 22) && !mbar_try_wait(bars + 8 * (t % NSTAGE), parity); ++spin) {}
            }
        }
    } else {
        cp_async_wait<0>();
    }
    __syncwarp();
}

__device__ __forceinline__ void load_q_frags(const Params &p, const __nv_bfloat16 *Q, int b, int i, int gkv, int lane,
                                             uint32_t (&qf)[16])
{
    const int g = lane >> 2, t = lane & 3;
    if (g < p.G) {
        const uint32_t *q = reinterpret_cast<const uint32_t *>(Q + b * p.qs_b + i * p.qs_t + (gkv * p.G + g) * p.qs_h);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qf[2 * ks] = __ldg(q + ks * 8 + t);
            qf[2 * ks + 1] = __ldg(q + ks * 8 + 4 + t);
        }
    } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) qf[e] = 0u;
    }
}

__device__ __forceinline__ void init_acc(Acc &acc, const Params &p, const float *sink, int gkv, int lane, bool with_sink)
{
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) acc.o[dt][0] = acc.o[dt][1] = acc.o[dt][2] = acc.o[dt][3] = 0.f;
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        const int head = 2 * t + hh;
        float m = -INFINITY;
        if (with_sink && sink && head < p.G) m = sink[gkv * p.G + head] * kLog2e;
        acc.m[hh] = m;
        acc.l[hh] = (m != -INFINITY && g == 0) ? 1.f : 0.f;   // e^{sink - m} = 1, counted once
    }
}

__device__ __forceinline__ void reduce_l(Acc &acc)
{
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        acc.l[hh] += __shfl_xor_sync(0xffffffffu, acc.l[hh], 4);
        acc.l[hh] += __shfl_xor_sync(0xffffffffu, acc.l[hh], 8);
        acc.l[hh] += __shfl_xor_sync(0xffffffffu, acc.l[hh], 16);
    }
}

// Normalise and store one (query, KV head) result: O rows of the G heads (16-byte stores, staged
// through the warp's shared memory) and LSE.
__device__ __forceinline__ void store_output(const Params &p, const Acc &acc, __nv_bfloat16 *O, float *LSE, int b, int i,
                                             int gkv, char *wsm, int lane)
{
    const int g = lane >> 2, t = lane & 3;
    constexpr int kPitch = HD + 8;   // bf16 elements per staged head row (bank spread)
    __nv_bfloat16 *so = reinterpret_cast<__nv_bfloat16 *>(wsm);
    float inv[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) inv[hh] = acc.l[hh] > 0.f ? 1.f / acc.l[hh] : 0.f;
#pragma unroll
    for (int dt = 0; dt < 8; ++dt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int head = 2 * t + (e & 1), d = 16 * dt + g + 8 * (e >> 1);
            so[head * kPitch + d] = __float2bfloat16_rn(acc.o[dt][e] * inv[e & 1]);
        }
    __syncwarp();
#pragma unroll
    for (int v = lane; v < 8 * 16; v += 32) {
        const int head = v >> 4, c = v & 15;
        if (head < p.G) {
            uint4 val = *reinterpret_cast<const uint4 *>(so + head * kPitch + c * 8);
            const int64_t off = b * p.os_b + i * p.os_t + (gkv * p.G + head) * p.os_h + c * 8;
            if (p.gate) {   // output gate: applied to the staged bf16 values, 8 at a time
                const uint4 gv = *reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(p.gate) + off);
                __nv_bfloat162 *ov = reinterpret_cast<__nv_bfloat162 *>(&val);
                const __nv_bfloat162 *gg = reinterpret_cast<const __nv_bfloat162 *>(&gv);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 o2 = __bfloat1622float2(ov[e]), g2 = __bfloat1622float2(gg[e]);
                    ov[e] = __floats2bfloat162_rn(o2.x * gate_of(g2.x), o2.y * gate_of(g2.y));
                }
            }
            *reinterpret_cast<uint4 *>(O + off) = val;
        }
    }
    if (LSE && g == 0) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int head = 2 * t + hh;
            if (head < p.G)
                LSE[((int64_t)b * p.Hq + gkv * p.G + head) * p.Lq + i] =
                    acc.l[hh] > 0.f ? (acc.m[hh] + log2f(acc.l[hh])) * kLn2 : -INFINITY;
        }
    }
    __syncwarp();
}

__device__ __forceinline__ Item make_item(const Params &p, const __nv_bfloat16 *K, const __nv_bfloat16 *V,
                                          const int32_t *idx, int b, int gkv, int i)
{
    Item it;
    // a group of 16 query heads runs as two sub-groups of 8: slot gkv of p.Hkv slots reads real KV head gkv / share
    const int share = p.share > 1 ? p.share : 1;
    const int g_real = gkv / share, hkv_real = p.Hkv / share;
    const int64_t base = b * p.ks_b + g_real * p.ks_h;
    it.Kb = reinterpret_cast<const char *>(K + base);
    it.Vb = reinterpret_cast<const char *>(V + base);
    it.row_stride = p.ks_t * 2;
    it.irow = idx ? idx + (((int64_t)b * hkv_real + g_real) * p.Lq + i) * p.k : nullptr;
    it.pos = pos_of(p, b, i);
    it.kvl = kvlen_of(p, b);
    it.raw = nullptr;
    it.lk = p.Lk;
    return it;
}

// ---------------------------------------------------------------- prefill: one warp per (b, g, i)
template <class C>
__global__ void __launch_bounds__(C::WARPS * 32)
k_sparse_prefill(const Params p, const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                 const __nv_bfloat16 *__restrict__ V, const int32_t *__restrict__ idx, const float *__restrict__ sink,
                 __nv_bfloat16 *__restrict__ O, float *__restrict__ LSE)
{
    extern __shared__ __align__(128) char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t item = (int64_t)blockIdx.x * C::WARPS + warp;   // (b, g, i), i fastest
    if (item >= (int64_t)p.B * p.Hkv * p.Lq) return;
    const int i = (int)(item % p.Lq);
    const int gkv = (int)((item / p.Lq) % p.Hkv);
    const int b = (int)(item / ((int64_t)p.Lq * p.Hkv));
    char *wsm = smem + warp * C::kWarpSmem;
    const Item it = make_item(p, K, V, idx, b, gkv, i);
    uint32_t qf[16];
    load_q_frags(p, Q, b, i, gkv, lane, qf);
    Acc acc;
    init_acc(acc, p, sink, gkv, lane, true);
    const int n_tiles = (p.k + p.w + C::KT - 1) / C::KT;
    run_tiles<C>(p, it, qf, acc, 0, n_tiles, wsm, lane);
    reduce_l(acc);
    store_output(p, acc, O, LSE, b, i, gkv, wsm, lane);
}

// ---------------------------------------------------------------- decode
// (a) enough (sequence, KV head) pairs to fill the GPU: one CTA per pair, its warps are the splits,
//     merged through shared memory.  No scratch, no atomics.
template <class C>
__global__ void __launch_bounds__(C::WARPS * 32)
k_sparse_decode_cta(const Params p, const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                    const __nv_bfloat16 *__restrict__ V, const int32_t *__restrict__ idx,
                    const float *__restrict__ sink, __nv_bfloat16 *__restrict__ O, float *__restrict__ LSE,
                    float *__restrict__ raw)
{
    extern __shared__ __align__(128) char smem[];
    constexpr int W = C::WARPS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int bg = blockIdx.x;
    const int gkv = bg % p.Hkv, b = bg / p.Hkv;
    const int g = lane >> 2, t = lane & 3;
    char *wsm = smem + warp * C::kWarpSmem;
    float *sml = reinterpret_cast<float *>(smem + W * C::kWarpSmem);   // [W][16]: m then l per head
    Item it = make_item(p, K, V, idx, b, gkv, 0);
    if (raw) it.raw = raw + (int64_t)bg * p.G * p.Lk;
    uint32_t qf[16];
    load_q_frags(p, Q, b, 0, gkv, lane, qf);
    Acc acc;
    init_acc(acc, p, sink, gkv, lane, warp == 0);   // the sink joins the denominator once
    const int n_tiles = (p.k + p.w + C::KT - 1) / C::KT;
    const int per = (n_tiles + W - 1) / W;
    run_tiles<C>(p, it, qf, acc, warp * per, min(n_tiles, (warp + 1) * per), wsm, lane);
    reduce_l(acc);
    float4 *op = reinterpret_cast<float4 *>(wsm);   // the warp's own staging area: [8][32] float4
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) op[dt * 32 + lane] = make_float4(acc.o[dt][0], acc.o[dt][1], acc.o[dt][2], acc.o[dt][3]);
    if (g == 0) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) { sml[warp * 16 + 2 * t + hh] = acc.m[hh]; sml[warp * 16 + 8 + 2 * t + hh] = acc.l[hh]; }
    }
    __syncthreads();
    if (warp != 0) return;
    Acc tot;
    float wgt[W][2];
    tot.m[0] = tot.m[1] = -INFINITY;
#pragma unroll
    for (int s = 0; s < W; ++s)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) tot.m[hh] = fmaxf(tot.m[hh], sml[s * 16 + 2 * t + hh]);
    tot.l[0] = tot.l[1] = 0.f;
#pragma unroll
    for (int s = 0; s < W; ++s)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const float ms = sml[s * 16 + 2 * t + hh];
            wgt[s][hh] = ms == -INFINITY ? 0.f : exp2f(ms - tot.m[hh]);
            tot.l[hh] += wgt[s][hh] * sml[s * 16 + 8 + 2 * t + hh];
        }
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s = 0; s < W; ++s) {
            const float4 v = reinterpret_cast<const float4 *>(smem + s * C::kWarpSmem)[dt * 32 + lane];
            a.x += wgt[s][0] * v.x; a.y += wgt[s][1] * v.y; a.z += wgt[s][0] * v.z; a.w += wgt[s][1] * v.w;
        }
        tot.o[dt][0] = a.x; tot.o[dt][1] = a.y; tot.o[dt][2] = a.z; tot.o[dt][3] = a.w;
    }
    __syncwarp();
    // the output staging must not overlap partials: it goes behind the per-warp areas
    store_output(p, tot, O, LSE, b, 0, gkv, smem + W * C::kWarpSmem + W * 16 * 4, lane);
}

// (b) few pairs: one warp per (pair, split); every warp publishes an un-normalised partial to global
//     scratch and the last one to arrive at the pair's ticket merges.  Nobody waits for anybody.
struct DecodeWs {
    int *tickets;     // [B * Hkv]
    float *ml;        // [items][2][8]   m then l per head
    float4 *opart;    // [items][8][32]  o[dt] of every lane
};

template <class C>
__global__ void __launch_bounds__(C::WARPS * 32)
k_sparse_decode_split(const Params p, const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                      const __nv_bfloat16 *__restrict__ V, const int32_t *__restrict__ idx,
                      const float *__restrict__ sink, __nv_bfloat16 *__restrict__ O, float *__restrict__ LSE,
                      DecodeWs ws, int n_splits, int tiles_per_split, float *__restrict__ raw)
{
    extern __shared__ __align__(128) char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t item = (int64_t)blockIdx.x * C::WARPS + warp;   // (b, g, split), split fastest
    if (item >= (int64_t)p.B * p.Hkv * n_splits) return;
    const int split = (int)(item % n_splits);
    const int bg = (int)(item / n_splits);
    const int gkv = bg % p.Hkv, b = bg / p.Hkv;
    const int g = lane >> 2, t = lane & 3;
    char *wsm = smem + warp * C::kWarpSmem;
    Item it = make_item(p, K, V, idx, b, gkv, 0);
    if (raw) it.raw = raw + (int64_t)bg * p.G * p.Lk;
    uint32_t qf[16];
    load_q_frags(p, Q, b, 0, gkv, lane, qf);
    Acc acc;
    init_acc(acc, p, sink, gkv, lane, split == 0);
    const int n_tiles = (p.k + p.w + C::KT - 1) / C::KT;
    const int t0 = split * tiles_per_split;
    run_tiles<C>(p, it, qf, acc, t0, min(n_tiles, t0 + tiles_per_split), wsm, lane);
    reduce_l(acc);
    float4 *op = ws.opart + item * 8 * 32;
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) op[dt * 32 + lane] = make_float4(acc.o[dt][0], acc.o[dt][1], acc.o[dt][2], acc.o[dt][3]);
    if (g == 0) {
        float *ml = ws.ml + item * 16;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) { ml[2 * t + hh] = acc.m[hh]; ml[8 + 2 * t + hh] = acc.l[hh]; }
    }
    __threadfence();
    __syncwarp();
    int ticket = 0;
    if (lane == 0) ticket = atomicAdd(ws.tickets + bg, 1);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    if (ticket != n_splits - 1) return;   // a later arrival merges
    __threadfence();
    const int64_t first = (int64_t)bg * n_splits;
    Acc tot;
    tot.m[0] = tot.m[1] = -INFINITY;
    for (int s = 0; s < n_splits; ++s) {
        const float *ml = ws.ml + (first + s) * 16;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) tot.m[hh] = fmaxf(tot.m[hh], __ldcg(ml + 2 * t + hh));
    }
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) tot.o[dt][0] = tot.o[dt][1] = tot.o[dt][2] = tot.o[dt][3] = 0.f;
    tot.l[0] = tot.l[1] = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        const float *ml = ws.ml + (first + s) * 16;
        float wgt[2];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const float ms = __ldcg(ml + 2 * t + hh);
            wgt[hh] = ms == -INFINITY ? 0.f : exp2f(ms - tot.m[hh]);
            tot.l[hh] += wgt[hh] * __ldcg(ml + 8 + 2 * t + hh);
        }
        const float4 *ops = ws.opart + (first + s) * 8 * 32;
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
            const float4 v = __ldcg(ops + dt * 32 + lane);
            tot.o[dt][0] += wgt[0] * v.x; tot.o[dt][1] += wgt[1] * v.y;
            tot.o[dt][2] += wgt[0] * v.z; tot.o[dt][3] += wgt[1] * v.w;
        }
    }
    store_output(p, tot, O, LSE, b, 0, gkv, wsm, lane);
}

size_t ws_tickets_bytes(const Params &p) { return ((size_t)p.B * p.Hkv * sizeof(int) + 255) / 256 * 256; }

constexpr int kDecodeCtaSmem = DecodeCfg::WARPS * DecodeCfg::kWarpSmem + DecodeCfg::WARPS * 16 * 4 + 8 * (HD + 8) * 2;

// SM count per device ordinal (0 = not asked yet); relaxed atomics: concurrent first calls write the same value
std::atomic<int> g_sm_count[64];
cudaError_t sm_count(int *n)
{
    int dev = 0, v = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool cached = dev >= 0 && dev < 64;
    if (cached && (v = g_sm_count[dev].load(std::memory_order_relaxed)) > 0) {
        *n = v;
        return cudaSuccess;
    }
    e = cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (cached) g_sm_count[dev].store(v, std::memory_order_relaxed);
    *n = v;
    return cudaSuccess;
}

// the opt-in to large dynamic shared memory is a per-device attribute of each kernel
bool g_attr_set[64] = {};
cudaError_t set_attrs()
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && g_attr_set[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(k_sparse_prefill<PrefillCfg>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             PrefillCfg::WARPS * PrefillCfg::kWarpSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_sparse_decode_split<DecodeCfg>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             DecodeCfg::WARPS * DecodeCfg::kWarpSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_sparse_decode_cta<DecodeCfg>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeCtaSmem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) g_attr_set[dev] = true;
    return cudaSuccess;
}

}  // namespace

bool sparse_mma_supported(const Params &p, hs2_dtype dt)
{
    auto m8 = [](int64_t x) { return x % 8 == 0; };
    if (p.ks_t * 2 > 0x7fffffffLL) return false;   // the row stride is used as a 32-bit multiplier
    return dt == HS2_BF16 && p.D == HD && p.G >= 1 && p.G <= 8 && m8(p.qs_b) && m8(p.qs_t) && m8(p.qs_h) &&
           m8(p.ks_b) && m8(p.ks_t) && m8(p.ks_h) && m8(p.os_b) && m8(p.os_t) && m8(p.os_h);
}

cudaError_t launch_sparse_mma_prefill(const Params &p, const void *Q, const void *K, const void *V, const int32_t *idx,
                                      const float *sink, void *O, float *LSE, cudaStream_t st)
{
    using C = PrefillCfg;
    cudaError_t e = set_attrs();
    if (e != cudaSuccess) return e;
    const int64_t items = (int64_t)p.B * p.Hkv * p.Lq;
    const unsigned blocks = (unsigned)((items + C::WARPS - 1) / C::WARPS);
    k_sparse_prefill<C><<<blocks, C::WARPS * 32, C::WARPS * C::kWarpSmem, st>>>(
        p, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, idx, sink, (__nv_bfloat16 *)O, LSE);
    count_launch();
    return cudaGetLastError();
}

size_t sparse_mma_decode_ws_bytes(const Params &p)
{
    const size_t items = (size_t)p.B * p.Hkv * kMaxSplits;
    return ws_tickets_bytes(p) + items * 16 * sizeof(float) + items * 8 * 32 * sizeof(float4);
}

cudaError_t launch_sparse_mma_decode(const Params &p, const void *Q, const void *K, const void *V, const int32_t *idx,
                                     const float *sink, void *O, float *LSE, void *ws, size_t ws_bytes, cudaStream_t st,
                                     float *raw)
{
    using C = DecodeCfg;
    cudaError_t e = set_attrs();
    if (e != cudaSuccess) return e;
    int sms = 0;
    if ((e = sm_count(&sms)) != cudaSuccess) return e;
    const int bg = p.B * p.Hkv;
    const int n_tiles = (p.k + p.w + C::KT - 1) / C::KT;
    const __nv_bfloat16 *q = (const __nv_bfloat16 *)Q, *k = (const __nv_bfloat16 *)K, *v = (const __nv_bfloat16 *)V;
    bool cta_path = bg >= sms && n_tiles >= 2 * C::WARPS;
#ifdef HS2_SP_SPLITS
    cta_path = false;   // tuning builds only
#endif
    if (cta_path) {
        k_sparse_decode_cta<C><<<bg, C::WARPS * 32, kDecodeCtaSmem, st>>>(p, q, k, v, idx, sink, (__nv_bfloat16 *)O, LSE, raw);
        count_launch();
    return cudaGetLastError();
    }
    // as many splits as fill every warp slot of the GPU once, each split at least two tiles long
    const int ctas_per_sm = (227 * 1024) / (C::WARPS * C::kWarpSmem) > 0 ? (227 * 1024) / (C::WARPS * C::kWarpSmem) : 1;
    int n_splits = (sms * ctas_per_sm * C::WARPS) / bg;
#ifdef HS2_SP_SPLITS
    n_splits = HS2_SP_SPLITS;
#endif
    n_splits = n_splits < 1 ? 1 : (n_splits > kMaxSplits ? kMaxSplits : n_splits);
    if (n_splits > (n_tiles + 1) / 2) n_splits = (n_tiles + 1) / 2 > 0 ? (n_tiles + 1) / 2 : 1;
    const int tiles_per_split = (n_tiles + n_splits - 1) / n_splits;
    n_splits = (n_tiles + tiles_per_split - 1) / tiles_per_split;
    if (n_splits <= 1) return raw ? cudaErrorNotSupported : launch_sparse_mma_prefill(p, Q, K, V, idx, sink, O, LSE, st);
    DecodeWs w;
    char *base = (char *)ws;
    const size_t items = (size_t)bg * kMaxSplits;
    w.tickets = (int *)base;
    w.ml = (float *)(base + ws_tickets_bytes(p));
    w.opart = (float4 *)(base + ws_tickets_bytes(p) + items * 16 * sizeof(float));
    (void)ws_bytes;
    if ((e = cudaMemsetAsync(w.tickets, 0, (size_t)bg * sizeof(int), st)) != cudaSuccess) return e;
    const int64_t n_items = (int64_t)bg * n_splits;
    const unsigned blocks = (unsigned)((n_items + C::WARPS - 1) / C::WARPS);
    k_sparse_decode_split<C><<<blocks, C::WARPS * 32, C::WARPS * C::kWarpSmem, st>>>(
        p, q, k, v, idx, sink, (__nv_bfloat16 *)O, LSE, w, n_splits, tiles_per_split, raw);
    count_launch();
    return cudaGetLastError();
}

// ---------------------------------------------------------------- selection scores from the kept raw products
// a[j] = max over the heads h of the group of (scale * raw[h][j] - LSE_h)   (Section 3.4); a thread takes four
// consecutive keys (one 16-byte load per head, several heads in flight) when the rows allow it, one key otherwise
template <bool VEC>
__global__ void __launch_bounds__(256)
k_scores_from_raw(const Params p, const float *__restrict__ raw, const float *__restrict__ LSE, float *__restrict__ out,
                  int64_t out_stride)
{
    const int bg = blockIdx.y;
    const int gkv = bg % p.Hkv, b = bg / p.Hkv;
    const float *lse = LSE + (int64_t)b * p.Hq + gkv * p.G;   // Lq == 1
    if (VEC) {
        const int j = (blockIdx.x * 256 + threadIdx.x) * 4;
        if (j >= p.Lk) return;
        const float *r = raw + (int64_t)bg * p.G * p.Lk + j;
        float4 a = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
#pragma unroll 4
        for (int h = 0; h < p.G; ++h) {
            const float4 v = __ldcs(reinterpret_cast<const float4 *>(r + (int64_t)h * p.Lk));
            const float nl = -lse[h];
            a.x = fmaxf(a.x, fmaf(p.scale, v.x, nl)); a.y = fmaxf(a.y, fmaf(p.scale, v.y, nl));
            a.z = fmaxf(a.z, fmaf(p.scale, v.z, nl)); a.w = fmaxf(a.w, fmaf(p.scale, v.w, nl));
        }
        *reinterpret_cast<float4 *>(out + (int64_t)bg * out_stride + j) = a;
    } else {
        const int j = blockIdx.x * 256 + threadIdx.x;
        if (j >= p.Lk) return;
        const float *r = raw + (int64_t)bg * p.G * p.Lk + j;
        float a = -INFINITY;
        for (int h = 0; h < p.G; ++h) a = fmaxf(a, fmaf(p.scale, r[(int64_t)h * p.Lk], -lse[h]));
        out[(int64_t)bg * out_stride + j] = a;
    }
}

cudaError_t launch_scores_from_raw(const Params &p, const float *raw, const float *LSE, float *out, int64_t out_stride,
                                   cudaStream_t st)
{
    const int bg = p.B * p.Hkv;
    if (bg <= 0 || bg > 65535 || p.Lq != 1) return cudaErrorNotSupported;
    const bool vec = p.Lk % 4 == 0 && out_stride % 4 == 0 && (reinterpret_cast<uintptr_t>(raw) & 15u) == 0 &&
                     (reinterpret_cast<uintptr_t>(out) & 15u) == 0;
    if (vec) {
        dim3 grid((unsigned)((p.Lk / 4 + 255) / 256), (unsigned)bg);
        k_scores_from_raw<true><<<grid, 256, 0, st>>>(p, raw, LSE, out, out_stride);
    } else {
        dim3 grid((unsigned)((p.Lk + 255) / 256), (unsigned)bg);
        k_scores_from_raw<false><<<grid, 256, 0, st>>>(p, raw, LSE, out, out_stride);
    }
    count_launch();
    return cudaGetLastError();
}

// ---------------------------------------------------------------- decode without caller scratch
// The split kernel above, with its partials and tickets in a fixed array that lives in the library
// image instead of a caller buffer.  Every device that loads the library carries the array until the
// process exits; all calls on a device share it.
namespace {

constexpr size_t kStaticTicketBytes = 256;
constexpr size_t kStaticItems = (size_t)kStaticDecodeMaxPairs * kMaxSplits;
constexpr size_t kStaticMlBytes = kStaticItems * 16 * sizeof(float);
constexpr size_t kStaticOpartBytes = kStaticItems * 8 * 32 * sizeof(float4);
constexpr size_t kStaticScratchBytes = kStaticTicketBytes + kStaticMlBytes + kStaticOpartBytes;   // 8,519,936 bytes
static_assert(kStaticDecodeMaxPairs * sizeof(int) <= kStaticTicketBytes, "tickets fit their slot");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void *g_static_scratch_addr[kMaxDevices] = {};   // device address of the array, per device ordinal
std::mutex g_static_mu;

// In host code `g_static_scratch` is only a handle; the address a kernel may use has to be asked
// for, once per device and with that device current.
cudaError_t static_scratch_address(void **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_scratch_addr[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress((void **)&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (!ptr) return cudaErrorInvalidSymbol;
        g_static_scratch_addr[dev] = ptr;
    }
    *out = g_static_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

bool sparse_mma_decode_static_fits(const Params &p) { return (int64_t)p.B * p.Hkv <= kStaticDecodeMaxPairs; }

cudaError_t launch_sparse_mma_decode_static(const Params &p, const void *Q, const void *K, const void *V,
                                            const int32_t *idx, const float *sink, void *O, float *LSE, cudaStream_t st)
{
    using C = DecodeCfg;
    cudaError_t e = set_attrs();
    if (e != cudaSuccess) return e;
    int sms = 0;
    if ((e = sm_count(&sms)) != cudaSuccess) return e;
    void *scratch = nullptr;
    if ((e = static_scratch_address(&scratch)) != cudaSuccess) return e;
    const int bg = p.B * p.Hkv;
    const int n_tiles = (p.k + p.w + C::KT - 1) / C::KT;
    const int ctas_per_sm = (227 * 1024) / (C::WARPS * C::kWarpSmem) > 0 ? (227 * 1024) / (C::WARPS * C::kWarpSmem) : 1;
    int n_splits = (sms * ctas_per_sm * C::WARPS) / bg;
    n_splits = n_splits < 1 ? 1 : (n_splits > kMaxSplits ? kMaxSplits : n_splits);
    if (n_splits > (n_tiles + 1) / 2) n_splits = (n_tiles + 1) / 2 > 0 ? (n_tiles + 1) / 2 : 1;
    const int tiles_per_split = (n_tiles + n_splits - 1) / n_splits;
    n_splits = (n_tiles + tiles_per_split - 1) / tiles_per_split;
    DecodeWs w;
    char *base = (char *)scratch;
    w.tickets = (int *)base;
    w.ml = (float *)(base + kStaticTicketBytes);
    w.opart = (float4 *)(base + kStaticTicketBytes + kStaticMlBytes);
    // the array keeps whatever the previous call left: the tickets must start at zero
    if ((e = cudaMemsetAsync(w.tickets, 0, (size_t)bg * sizeof(int), st)) != cudaSuccess) return e;
    const int64_t n_items = (int64_t)bg * n_splits;
    const unsigned blocks = (unsigned)((n_items + C::WARPS - 1) / C::WARPS);
    k_sparse_decode_split<C><<<blocks, C::WARPS * 32, C::WARPS * C::kWarpSmem, st>>>(
        p, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, idx, sink, (__nv_bfloat16 *)O, LSE,
        w, n_splits, tiles_per_split, nullptr);
    count_launch();
    return cudaGetLastError();
}

// device error word of the sparse kernels (bit 0: a bounded wait ran out); synchronises the device
cudaError_t read_sparse_error(unsigned *out) { return cudaMemcpyFromSymbol(out, g_sparse_error, sizeof(unsigned)); }

}  // namespace hs2
