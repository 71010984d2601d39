// Sparse attention over (reused top-k indices) U (forced window) on an FP8 KV cache: K and V stored as e4m3
// codes with one fp32 scale per (token, KV head); Q and O stay bf16; head_dim 128, group <= 8.
// (Section 3.3 for the operator; the paper's cost analysis of Section 4 assumes FP8 KV-cache storage.)
//
// The gather is bound by memory, so halving the bytes of a row is the whole point: a K or V row is 128 bytes
// (+ 4 bytes of scale).  Structure as in the bf16 gather kernel - one warp per (query, KV head) item with a
// private cp.async pipeline, keys on the MMA M dimension, heads on N - with these differences:
//   * the stage holds the raw e4m3 rows (128-byte rows, 16-byte chunks XOR-swizzled by the row);
//   * ldmatrix moves 16-bit units, i.e. PAIRS of codes.  For S^T = K Q^T a thread therefore receives four
//     consecutive dims of a key per register; they are converted to two f16x2 registers (cvt e4m3x2 -> f16x2,
//     exact) and used as k-slots (2t, 2t+1) and (2t+8, 2t+9) of an m16n8k16 f16 MMA - a permutation of the
//     contraction index, matched by loading Q in the same order (four consecutive dims per thread);
//   * for O^T = V^T P^T the transposing ldmatrix delivers, per register, codes (key 2t, dims 2g, 2g+1) and
//     (key 2t+1, dims 2g, 2g+1); one byte permute makes them (dim 2g: keys 2t, 2t+1 | dim 2g+1: keys 2t, 2t+1),
//     so MMA row g is dim 2g and row g+8 is dim 2g+1 of a 16-dim slice: the accumulator's dim order is a
//     permutation that only the final store has to know;
//   * the scales never touch the operands: the K scale multiplies the score row of its key, the V scale is
//     folded into the probability of its key (times 2^8 to stay inside the normal range of f16; undone in the
//     store).  The denominator sums the unscaled probabilities.
// Prefill: one buffer of 32 rows per warp (fetch, wait, fold) and 16 warps per SM, as in the bf16 kernel - whose
// warps need twice the shared memory, so that only 12 of them fit.  Decode: one CTA per (sequence, KV head), its
// warps split the attended set (two stages of 16 rows each) and merge through shared memory; with a pointer for them
// it also leaves the dequantised q.k of every (head, key) behind, for the selection of the full layer's decode step.
#include <cuda_fp16.h>

#include "hs2_common.cuh"

#ifndef HS2_F8_WARPS
#define HS2_F8_WARPS 16
#endif
#ifndef HS2_F8D_WARPS
#define HS2_F8D_WARPS 8
#endif
#ifndef HS2_F8D_MINB
#define HS2_F8D_MINB 2
#endif

namespace hs2 {
namespace {

constexpr int HD = 128;
#ifndef HS2_F8_KT
#define HS2_F8_KT 16
#endif
#ifndef HS2_F8_PKT
#define HS2_F8_PKT 32
#endif
constexpr int KTD = HS2_F8_KT;               // key rows per stage, decode (32-row stages were measured: 47.8 vs 45.3 us per step)
constexpr int KTP = HS2_F8_PKT;              // key rows per buffer, prefill
static_assert((KTD == 16 || KTD == 32) && (KTP == 16 || KTP == 32), "a stage holds 16 or 32 key rows");
#ifndef HS2_F8_NSTAGE
#define HS2_F8_NSTAGE 2
#endif
#ifndef HS2_F8_PNSTAGE
#define HS2_F8_PNSTAGE 1    // stages per warp in the prefill kernel (one buffer of 32 rows and 16 warps measured best)
#endif
constexpr int NSTAGE = HS2_F8_NSTAGE;
constexpr int kRow = HD;                     // bytes of one e4m3 row
// a stage of KT rows: the K tile, the V tile; per stage also: key index of each row (32 ints), K scales (KT), V scales (KT)
template <int KT> struct Stage {
    static constexpr int MT = KT / 16;               // 16-key MMA tiles per stage
    static constexpr int kTile = KT * kRow;          // one K or V tile
    static constexpr int kStageBytes = 2 * kTile;
    static constexpr int kMetaBytes = 32 * 4 + 2 * KT * 4;
};
constexpr int kWarpSmem = NSTAGE * (Stage<KTD>::kStageBytes + Stage<KTD>::kMetaBytes);   // decode
constexpr int NSP = HS2_F8_PNSTAGE;
constexpr int kWarpSmemP = NSP * (Stage<KTP>::kStageBytes + Stage<KTP>::kMetaBytes);     // prefill
constexpr float kPShift = 256.f;             // probabilities x V scale are carried x 2^8 through the f16 operand

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }
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
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// two e4m3 codes (low byte first) -> f16x2 (low half first); exact
__device__ __forceinline__ uint32_t cvt_e4m3x2(uint32_t two_codes)
{
    uint32_t d;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;\n" : "=r"(d) : "h"((unsigned short)two_codes));
    return d;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi)
{
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Accumulators of one warp.  Thread (g = lane/4, t = lane%4) owns heads 2t and 2t+1 of the group:
// o[dt][0..3] = O^T at (dim 16 dt + 2g, head 2t), (same dim, head 2t+1), (dim 16 dt + 2g + 1, head 2t),
// (dim 16 dt + 2g + 1, head 2t+1), all times 2^8; m is replicated over g, l is this thread's partial sum.
struct Acc {
    float o[8][4];
    float m[2], l[2];
};

struct Item {
    const char *Kb, *Vb;          // first row of this (sequence, KV head)
    const float *ksc, *vsc;       // its scales: element j * Hkv
    int64_t row_stride;           // bytes between consecutive tokens
    int64_t sc_stride;            // floats between consecutive tokens' scales
    const int32_t *irow;
    int pos, kvl;
    float *raw;                   // decode-shaped full layer: dequantised q.k of every (head, key) goes here, or null
    int lk;
};

__device__ __forceinline__ Item make_item(const Params &p, const uint8_t *K, const uint8_t *V, const float *ksc, const float *vsc,
                                          const int32_t *idx, int b, int gkv, int i)
{
    Item it;
    // a group of 16 query heads runs as two sub-groups of 8: slot gkv of p.Hkv slots reads real KV head gkv / share
    const int share = p.share > 1 ? p.share : 1;
    const int g_real = gkv / share, hkv_real = p.Hkv / share;
    const int64_t base = b * p.ks_b + g_real * p.ks_h;
    it.Kb = reinterpret_cast<const char *>(K + base);
    it.Vb = reinterpret_cast<const char *>(V + base);
    it.ksc = ksc + b * p.ss_b + g_real * p.ss_h;
    it.vsc = vsc + b * p.ss_b + g_real * p.ss_h;
    it.row_stride = p.ks_t;
    it.sc_stride = p.ss_t;
    it.irow = idx ? idx + (((int64_t)b * hkv_real + g_real) * p.Lq + i) * p.k : nullptr;
    it.pos = pos_of(p, b, i);
    it.kvl = kvlen_of(p, b);
    it.raw = nullptr;
    it.lk = 0;
    return it;
}

// Slot s of the virtual slot array [idx row | window] holds a key index or is void (-1).  slot_raw starts the fetch
// (an idx entry is a global load), slot_fix applies the validity rules when the value is used one tile later, so
// that the load's latency is never waited for.
template <int KT>
__device__ __forceinline__ int slot_raw(const Params &p, const Item &it, int tile, int lane)
{
    const int s = tile * KT + lane;
    if (lane >= KT) return -1;
    if (s < p.k) return it.irow ? __ldg(it.irow + s) : -1;
    return s < p.k + p.w ? it.pos - p.w + 1 + (s - p.k) : -1;
}
template <int KT>
__device__ __forceinline__ int slot_fix(const Params &p, const Item &it, int tile, int lane, int j)
{
    const int hi = tile * KT + lane < p.k ? it.pos - p.w : it.pos;   // idx entries inside the window are void
    return (j < 0 || j > hi || j >= it.kvl) ? -1 : j;
}

// lane -> 16-byte chunk c (of 8) of rows r0 + (lane >> 3); the lanes also fetch the stage's scales.  Void rows are
// zero filled, nothing is read for them.
template <int KT>
__device__ __forceinline__ void issue_stage(const Item &it, uint32_t stage_base, uint32_t meta_base, int j, int lane)
{
    constexpr int kTile = Stage<KT>::kTile;
    const int c = lane & 7, hi = lane >> 3;
    const char *kc = it.Kb + c * 16, *vc = it.Vb + c * 16;
#pragma unroll
    for (int r0 = 0; r0 < KT; r0 += 4) {
        const int r = r0 + hi;
        const int jr = __shfl_sync(0xffffffffu, j, r);
        const uint32_t dst = stage_base + r * kRow + ((uint32_t)(c ^ (r & 7)) << 4);
        const int64_t off = (int64_t)max(jr, 0) * it.row_stride;
        const int nbytes = jr < 0 ? 0 : 16;
        cp_async16(dst, kc + off, nbytes);
        cp_async16(dst + kTile, vc + off, nbytes);
    }
    // the 2 * KT scales of the stage: K scales of rows 0..KT-1, then V scales
#pragma unroll
    for (int s0 = 0; s0 < 2 * KT; s0 += 32) {
        const int sl = s0 + lane;
        const int js = __shfl_sync(0xffffffffu, j, sl % KT);
        const float *sp = (sl < KT ? it.ksc : it.vsc) + (int64_t)max(js, 0) * it.sc_stride;
        cp_async4(meta_base + 32 * 4 + sl * 4, sp, js < 0 ? 0 : 4);
    }
}

template <int KT>
__device__ __forceinline__ void consume_stage(Acc &acc, const uint32_t (&qf)[16], uint32_t stage_base, const float *sks,
                                              const float *svs, unsigned mask, float scale_log2, int lane,
                                              float *raw = nullptr, int lk = 0, int G = 0, const int *sjrow = nullptr)
{
    constexpr int MT = Stage<KT>::MT, kTile = Stage<KT>::kTile;
    const int g = lane >> 2;
    const int mi = lane >> 3, rr = lane & 7;
    float s[MT][4];
    // S^T = K Q^T : rows = keys, columns = heads.  One ldmatrix = 16 keys x 32 dims = two MMAs.
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        float s2[4] = {0.f, 0.f, 0.f, 0.f};
        s[mt][0] = s[mt][1] = s[mt][2] = s[mt][3] = 0.f;
        const uint32_t rowaddr = stage_base + (mt * 16 + (mi & 1) * 8 + rr) * kRow;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t a[4];
            ldmatrix_x4(a, rowaddr + ((uint32_t)((2 * q4 + (mi >> 1)) ^ rr) << 4));
            mma_f16(s[mt], cvt_e4m3x2(a[0]), cvt_e4m3x2(a[1]), cvt_e4m3x2(a[0] >> 16), cvt_e4m3x2(a[1] >> 16), qf[4 * q4], qf[4 * q4 + 1]);
            mma_f16(s2, cvt_e4m3x2(a[2]), cvt_e4m3x2(a[3]), cvt_e4m3x2(a[2] >> 16), cvt_e4m3x2(a[3] >> 16), qf[4 * q4 + 2], qf[4 * q4 + 3]);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) s[mt][e] += s2[e];
    }
    if (raw) {
        // The decode-shaped full layer keeps the dequantised products: the selection scores need the final LSE, and
        // reading them back (4 bytes per head and key) is far cheaper than sweeping K a second time.
        const int t = lane & 3;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int row = mt * 16 + g + 8 * r;
                const int j = sjrow[row];
                if (j >= 0) {
                    const float ks = sks[row];
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh)
                        if (2 * t + hh < G) raw[(int64_t)(2 * t + hh) * lk + j] = s[mt][2 * r + hh] * ks;
                }
            }
    }
    // dequantise the score rows, online softmax in the base-2 domain; this thread: heads 2t+hh, keys 16 mt + g + 8 r
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = mt * 16 + g + 8 * r;
            const bool ok = (mask >> row) & 1u;
            const float ks = sks[row] * scale_log2;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const float t2 = ok ? s[mt][2 * r + hh] * ks : -INFINITY;
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
    uint32_t pb[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        float pv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            pv[e] = exp2f(s[mt][e] - muse[e & 1]);
            acc.l[e & 1] += pv[e];
        }
        const float vs0 = svs[mt * 16 + g] * kPShift, vs1 = svs[mt * 16 + g + 8] * kPShift;
        pb[mt][0] = movmatrix_trans(pack_f16(pv[0] * vs0, pv[1] * vs0));   // keys 16 mt + 0..7
        pb[mt][1] = movmatrix_trans(pack_f16(pv[2] * vs1, pv[3] * vs1));   // keys 16 mt + 8..15
    }
    if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
            acc.o[dt][0] *= corr[0]; acc.o[dt][1] *= corr[1];
            acc.o[dt][2] *= corr[0]; acc.o[dt][3] *= corr[1];
        }
    }
    // O^T += V^T P^T : one transposing ldmatrix = 16 keys x 32 dims = two MMAs (16 dims each)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const uint32_t rowaddr = stage_base + kTile + (mt * 16 + (mi & 1) * 8 + rr) * kRow;
#pragma unroll
        for (int dq = 0; dq < 4; ++dq) {
            uint32_t a[4];
            ldmatrix_x4_trans(a, rowaddr + ((uint32_t)((2 * dq + (mi >> 1)) ^ rr) << 4));
#pragma unroll
            for (int e = 0; e < 4; ++e) a[e] = __byte_perm(a[e], 0u, 0x3120);   // (dim 2g: keys 2t, 2t+1 | dim 2g+1: keys 2t, 2t+1)
            mma_f16(acc.o[2 * dq], cvt_e4m3x2(a[0]), cvt_e4m3x2(a[0] >> 16), cvt_e4m3x2(a[1]), cvt_e4m3x2(a[1] >> 16), pb[mt][0], pb[mt][1]);
            mma_f16(acc.o[2 * dq + 1], cvt_e4m3x2(a[2]), cvt_e4m3x2(a[2] >> 16), cvt_e4m3x2(a[3]), cvt_e4m3x2(a[3] >> 16), pb[mt][0], pb[mt][1]);
        }
    }
}

// Fold slot tiles [t_begin, t_end) of one item into acc with an NS-deep cp.async pipeline.  NS = 1: fetch, wait, fold in
// one buffer; the warp overlaps nothing by itself, but needs half the shared memory, so more warps are resident.
template <int NS, int KT>
__device__ __forceinline__ void run_tiles(const Params &p, const Item &it, const uint32_t (&qf)[16], Acc &acc, int t_begin,
                                          int t_end, char *wsm, int lane)
{
    constexpr int kStageBytes = Stage<KT>::kStageBytes, kMetaBytes = Stage<KT>::kMetaBytes;
    const uint32_t sbase = smem_u32(wsm);
    char *meta = wsm + NS * kStageBytes;
    const uint32_t mbase = sbase + NS * kStageBytes;
    int next = t_begin;
    int jn = next < t_end ? slot_raw<KT>(p, it, next, lane) : -1;
    int n_issued = 0, n_done = 0;
    auto try_issue = [&](int stage) -> bool {
        while (next < t_end) {
            const int j = slot_fix<KT>(p, it, next, lane, jn);
            ++next;
            if (next < t_end) jn = slot_raw<KT>(p, it, next, lane);
            if (__ballot_sync(0xffffffffu, j >= 0)) {   // all-void tiles are skipped
                reinterpret_cast<int *>(meta + stage * kMetaBytes)[lane] = j;
                issue_stage<KT>(it, sbase + stage * kStageBytes, mbase + stage * kMetaBytes, j, lane);
                return true;
            }
        }
        return false;
    };
    if (NS == 1) {
        while (try_issue(0)) {
            cp_async_commit();
            cp_async_wait<0>();
            __syncwarp();
            const unsigned mask = __ballot_sync(0xffffffffu, reinterpret_cast<const int *>(meta)[lane] >= 0);
            consume_stage<KT>(acc, qf, sbase, reinterpret_cast<const float *>(meta + 32 * 4),
                          reinterpret_cast<const float *>(meta + 32 * 4 + KT * 4), mask, p.scale_log2, lane, it.raw, it.lk, p.G,
                          reinterpret_cast<const int *>(meta));
            __syncwarp();   // every lane has read the buffer before the next tile's copies land in it
        }
        return;
    }
#pragma unroll
    for (int s = 0; s < NS - 1; ++s) {
        if (try_issue(n_issued % NS)) ++n_issued;
        cp_async_commit();
    }
    while (n_done < n_issued) {
        const int stage = n_done % NS;
        cp_async_wait<(NS >= 2 ? NS - 2 : 0)>();
        __syncwarp();
        if (try_issue(n_issued % NS)) ++n_issued;
        cp_async_commit();
        const char *mt = meta + stage * kMetaBytes;
        const unsigned mask = __ballot_sync(0xffffffffu, reinterpret_cast<const int *>(mt)[lane] >= 0);
        consume_stage<KT>(acc, qf, sbase + stage * kStageBytes, reinterpret_cast<const float *>(mt + 32 * 4),
                      reinterpret_cast<const float *>(mt + 32 * 4 + KT * 4), mask, p.scale_log2, lane, it.raw, it.lk, p.G,
                      reinterpret_cast<const int *>(mt));
        ++n_done;
    }
    cp_async_wait<0>();
    __syncwarp();
}

// Q of head g in the contraction order of the K fragments: four consecutive dims per thread and 16-dim step.
__device__ __forceinline__ void load_q_frags(const Params &p, const __nv_bfloat16 *Q, int b, int i, int gkv, int lane,
                                             uint32_t (&qf)[16])
{
    const int g = lane >> 2, t = lane & 3;
    if (g < p.G) {
        const __nv_bfloat16 *q = Q + b * p.qs_b + i * p.qs_t + (gkv * p.G + g) * p.qs_h;
#pragma unroll
        for (int st = 0; st < 8; ++st) {   // dims 16 st + 4 t .. + 3
            const uint2 raw = __ldg(reinterpret_cast<const uint2 *>(q + 16 * st + 4 * t));
            const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.x));
            const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&raw.y));
            qf[2 * st] = pack_f16(lo.x, lo.y);
            qf[2 * st + 1] = pack_f16(hi.x, hi.y);
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
        acc.l[hh] = (m != -INFINITY && g == 0) ? 1.f : 0.f;
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

// Normalise and store one (query, KV head) result (staged through the warp's shared memory for 16-byte stores).
__device__ __forceinline__ void store_output(const Params &p, const Acc &acc, __nv_bfloat16 *O, float *LSE, int b, int i,
                                             int gkv, char *wsm, int lane)
{
    const int g = lane >> 2, t = lane & 3;
    constexpr int kPitchO = HD + 8;   // bf16 elements per staged head row
    __nv_bfloat16 *so = reinterpret_cast<__nv_bfloat16 *>(wsm);
    float inv[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) inv[hh] = acc.l[hh] > 0.f ? (1.f / kPShift) / acc.l[hh] : 0.f;
#pragma unroll
    for (int dt = 0; dt < 8; ++dt)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {   // dims 16 dt + 2g and + 1 of head 2t + hh are adjacent: one 4-byte store
            const uint32_t two = pack_bf16(acc.o[dt][hh] * inv[hh], acc.o[dt][2 + hh] * inv[hh]);
            *reinterpret_cast<uint32_t *>(so + (2 * t + hh) * kPitchO + 16 * dt + 2 * g) = two;
        }
    __syncwarp();
#pragma unroll
    for (int v = lane; v < 8 * 16; v += 32) {
        const int head = v >> 4, c = v & 15;
        if (head < p.G) {
            const uint4 val = *reinterpret_cast<const uint4 *>(so + head * kPitchO + c * 8);
            *reinterpret_cast<uint4 *>(O + b * p.os_b + i * p.os_t + (gkv * p.G + head) * p.os_h + c * 8) = val;
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
}

// ---------------------------------------------------------------- prefill: one warp per (b, g, i)
__global__ void __launch_bounds__(HS2_F8_WARPS * 32)
k_sparse_fp8_prefill(const Params p, const __nv_bfloat16 *__restrict__ Q, const uint8_t *__restrict__ K,
                     const uint8_t *__restrict__ V, const float *__restrict__ ksc, const float *__restrict__ vsc,
                     const int32_t *__restrict__ idx, const float *__restrict__ sink, __nv_bfloat16 *__restrict__ O,
                     float *__restrict__ LSE)
{
    extern __shared__ __align__(128) char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t item = (int64_t)blockIdx.x * HS2_F8_WARPS + warp;   // (b, g, i), i fastest
    if (item >= (int64_t)p.B * p.Hkv * p.Lq) return;
    const int i = (int)(item % p.Lq);
    const int gkv = (int)((item / p.Lq) % p.Hkv);
    const int b = (int)(item / ((int64_t)p.Lq * p.Hkv));
    char *wsm = smem + warp * kWarpSmemP;
    const Item it = make_item(p, K, V, ksc, vsc, idx, b, gkv, i);
    uint32_t qf[16];
    load_q_frags(p, Q, b, i, gkv, lane, qf);
    Acc acc;
    init_acc(acc, p, sink, gkv, lane, true);
    run_tiles<NSP, KTP>(p, it, qf, acc, 0, (p.k + p.w + KTP - 1) / KTP, wsm, lane);
    reduce_l(acc);
    store_output(p, acc, O, LSE, b, i, gkv, wsm, lane);
}

// ---------------------------------------------------------------- decode: one CTA per (sequence, KV head)
__global__ void __launch_bounds__(HS2_F8D_WARPS * 32, HS2_F8D_MINB)
k_sparse_fp8_decode(const Params p, const __nv_bfloat16 *__restrict__ Q, const uint8_t *__restrict__ K,
                    const uint8_t *__restrict__ V, const float *__restrict__ ksc, const float *__restrict__ vsc,
                    const int32_t *__restrict__ idx, const float *__restrict__ sink, __nv_bfloat16 *__restrict__ O,
                    float *__restrict__ LSE, float *__restrict__ raw)
{
    extern __shared__ __align__(128) char smem[];
    constexpr int W = HS2_F8D_WARPS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int bg = blockIdx.x;
    const int gkv = bg % p.Hkv, b = bg / p.Hkv;
    const int g = lane >> 2, t = lane & 3;
    char *wsm = smem + warp * kWarpSmem;
    float *sml = reinterpret_cast<float *>(smem + W * kWarpSmem);   // [W][16]: m then l per head
    Item it = make_item(p, K, V, ksc, vsc, idx, b, gkv, 0);
    if (raw) { it.raw = raw + (int64_t)bg * p.G * p.Lk; it.lk = p.Lk; }
    uint32_t qf[16];
    load_q_frags(p, Q, b, 0, gkv, lane, qf);
    Acc acc;
    init_acc(acc, p, sink, gkv, lane, warp == 0);   // the sink joins the denominator once
    const int n_tiles = (p.k + p.w + KTD - 1) / KTD;
    const int per = (n_tiles + W - 1) / W;
    run_tiles<NSTAGE, KTD>(p, it, qf, acc, warp * per, min(n_tiles, (warp + 1) * per), wsm, lane);
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
            const float4 v = reinterpret_cast<const float4 *>(smem + s * kWarpSmem)[dt * 32 + lane];
            a.x += wgt[s][0] * v.x; a.y += wgt[s][1] * v.y; a.z += wgt[s][0] * v.z; a.w += wgt[s][1] * v.w;
        }
        tot.o[dt][0] = a.x; tot.o[dt][1] = a.y; tot.o[dt][2] = a.z; tot.o[dt][3] = a.w;
    }
    __syncwarp();
    // the output staging must not overlap the partials: it goes behind the per-warp areas
    store_output(p, tot, O, LSE, b, 0, gkv, smem + W * kWarpSmem + W * 16 * 4, lane);
}

constexpr int kPrefillSmem = HS2_F8_WARPS * kWarpSmemP;
constexpr int kDecodeSmem = HS2_F8D_WARPS * kWarpSmem + HS2_F8D_WARPS * 16 * 4 + 8 * (HD + 8) * 2;
static_assert(NSTAGE * Stage<KTD>::kStageBytes >= 8 * 32 * 16, "a warp's stages hold its partial accumulator in decode");
static_assert(NSTAGE * Stage<KTD>::kStageBytes >= 8 * (HD + 8) * 2 && NSP * Stage<KTP>::kStageBytes >= 8 * (HD + 8) * 2,
              "a warp's stages hold its staged output rows");

template <class Kern>
cudaError_t set_smem(Kern kern, int bytes, bool *done)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorNotSupported;
    if (!done[dev]) {
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes)) != cudaSuccess) return e;
        done[dev] = true;
    }
    return cudaSuccess;
}

}  // namespace

// bf16 queries, e4m3 cache with a scale per (token, KV head): head_dim 128, group <= 8; strides in bytes for the cache
// ---------------------------------------------------------------- selection scores of a one-query layer on the FP8 cache
// a[j] = max over the heads h of the group of (scale * k_scale[j] * <q_h, code_j> - LSE_h)   (Section 3.4), for one
// query per sequence, any group of up to 128 heads, head_dim 128 or 256: the second pass of the full layer's decode step
// on shapes whose first pass (attention, LSE) runs on the tcgen05 gather kernel.  Memory-bound: every key's codes are
// read once.  A warp takes 16 consecutive keys against all heads: the key codes go from global memory straight into
// MMA A fragments (a thread reads 16 consecutive bytes of a row: four consecutive dims for each of four k-steps, a
// permutation of the contraction index that the query fragments in shared memory follow), cvt e4m3x2 -> f16x2 is exact.
namespace {

constexpr int kScF8Warps = 8;

template <int D>
__global__ void __launch_bounds__(kScF8Warps * 32)
k_scores_fp8_decode(const Params p, const __nv_bfloat16 *__restrict__ Q, const uint8_t *__restrict__ K,
                    const float *__restrict__ ksc, const float *__restrict__ LSE, float *__restrict__ out, int64_t out_stride)
{
    extern __shared__ __align__(16) unsigned char s_raw[];
    const int GP = (p.G + 7) & ~7, NT = GP / 8;                 // heads padded to whole n-tiles of 8
    uint2 *s_q = reinterpret_cast<uint2 *>(s_raw);              // [NT][D / 16 k-steps][32 lanes]: the B fragments
    float *s_lse = reinterpret_cast<float *>(s_raw + (size_t)NT * (D / 16) * 32 * 8);   // [GP], natural log; +inf past the group
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bg = blockIdx.y, gkv = bg % p.Hkv, b = bg / p.Hkv;
    const int g = lane >> 2, t = lane & 3;
    const int n_keys = max(0, min(pos_of(p, b, 0) - p.w + 1, kvlen_of(p, b)));
    // query fragments: n-tile nt, k-step ks = 4 c + i (c: 64-dim slice, i: word of the 16-byte run), lane (g, t):
    // b0 = dims (64 c + 16 t + 4 i, + 1), b1 = (+ 2, + 3) of head 8 nt + g
    for (int e = tid; e < NT * (D / 16) * 32; e += blockDim.x) {
        const int ln = e & 31, ks = (e >> 5) % (D / 16), nt = e / (32 * (D / 16));
        const int hg = ln >> 2, ht = ln & 3, c = ks >> 2, i = ks & 3;
        const int head = 8 * nt + hg;
        uint2 frag = make_uint2(0u, 0u);
        if (head < p.G) {
            const __nv_bfloat16 *q = Q + b * p.qs_b + (gkv * p.G + head) * p.qs_h + 64 * c + 16 * ht + 4 * i;
            const uint2 rawq = __ldg(reinterpret_cast<const uint2 *>(q));
            const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&rawq.x));
            const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&rawq.y));
            frag = make_uint2(pack_f16(lo.x, lo.y), pack_f16(hi.x, hi.y));
        }
        s_q[e] = frag;
    }
    for (int h = tid; h < GP; h += blockDim.x) s_lse[h] = h < p.G ? LSE[((int64_t)b * p.Hq + gkv * p.G + h) * p.Lq] : INFINITY;
    __syncthreads();
    float *orow = out + (int64_t)bg * out_stride;
    const uint8_t *kbase = K + b * p.ks_b + gkv * p.ks_h;
    const int64_t rs = p.ks_t;                                   // bytes between consecutive tokens
    const float *ksb = ksc + b * p.ss_b + gkv * p.ss_h;
    for (int j0 = (blockIdx.x * kScF8Warps + warp) * 16; j0 < n_keys; j0 += gridDim.x * kScF8Warps * 16) {
        const int ja = j0 + g, jb = j0 + g + 8;                  // this thread's two keys
        const bool va = ja < n_keys, vb = jb < n_keys;
        uint4 ca[D / 64], cb[D / 64];
#pragma unroll
        for (int c = 0; c < D / 64; ++c) {
            ca[c] = va ? __ldg(reinterpret_cast<const uint4 *>(kbase + (int64_t)ja * rs + 64 * c + 16 * t)) : make_uint4(0u, 0u, 0u, 0u);
            cb[c] = vb ? __ldg(reinterpret_cast<const uint4 *>(kbase + (int64_t)jb * rs + 64 * c + 16 * t)) : make_uint4(0u, 0u, 0u, 0u);
        }
        const float fa = va ? __ldg(ksb + (int64_t)ja * p.ss_t) * p.scale : 0.f;
        const float fb = vb ? __ldg(ksb + (int64_t)jb * p.ss_t) * p.scale : 0.f;
        float best_a = -INFINITY, best_b = -INFINITY;
        for (int nt = 0; nt < NT; ++nt) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            const uint2 *qf = s_q + (size_t)nt * (D / 16) * 32 + lane;
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                const uint32_t wa[4] = {ca[c].x, ca[c].y, ca[c].z, ca[c].w}, wb[4] = {cb[c].x, cb[c].y, cb[c].z, cb[c].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint2 bq = qf[(4 * c + i) * 32];
                    mma_f16(acc, cvt_e4m3x2(wa[i]), cvt_e4m3x2(wb[i]), cvt_e4m3x2(wa[i] >> 16), cvt_e4m3x2(wb[i] >> 16), bq.x, bq.y);
                }
            }
            // acc[0], acc[1]: key ja, heads 8 nt + 2 t, + 1; acc[2], acc[3]: key jb
            const float l0 = s_lse[8 * nt + 2 * t], l1 = s_lse[8 * nt + 2 * t + 1];
            best_a = fmaxf(best_a, fmaxf(acc[0] * fa - l0, acc[1] * fa - l1));
            best_b = fmaxf(best_b, fmaxf(acc[2] * fb - l0, acc[3] * fb - l1));
        }
        best_a = fmaxf(best_a, __shfl_xor_sync(0xffffffffu, best_a, 1));
        best_a = fmaxf(best_a, __shfl_xor_sync(0xffffffffu, best_a, 2));
        best_b = fmaxf(best_b, __shfl_xor_sync(0xffffffffu, best_b, 1));
        best_b = fmaxf(best_b, __shfl_xor_sync(0xffffffffu, best_b, 2));
        if (t == 0) {
            if (va) orow[ja] = best_a;
            if (vb) orow[jb] = best_b;
        }
    }
}

}  // namespace

// rows = (b, g), row stride out_stride floats; keys beyond a row's candidates are not written
cudaError_t launch_scores_fp8_decode(const Params &p, const void *Q, const void *K8, const float *ksc, const float *LSE,
                                     float *out, int64_t out_stride, cudaStream_t st)
{
    const int bg = p.B * p.Hkv;
    if (p.Lq != 1 || bg <= 0 || bg > 65535 || p.G > 128 || (p.D != 128 && p.D != 256)) return cudaErrorNotSupported;
    const int GP = (p.G + 7) & ~7;
    const size_t smem = (size_t)(GP / 8) * (p.D / 16) * 32 * 8 + (size_t)GP * 4;
    int gx = (p.Lk + kScF8Warps * 16 - 1) / (kScF8Warps * 16);
    const int cap = (148 * 8 + bg - 1) / bg;      // about eight CTAs per SM over the whole grid
    if (gx > cap) gx = cap < 1 ? 1 : cap;
    cudaError_t e = cudaSuccess;
    if (p.D == 128) {
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(k_scores_fp8_decode<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_scores_fp8_decode<128><<<dim3((unsigned)gx, (unsigned)bg), kScF8Warps * 32, smem, st>>>(
            p, (const __nv_bfloat16 *)Q, (const uint8_t *)K8, ksc, LSE, out, out_stride);
    } else {
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(k_scores_fp8_decode<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        k_scores_fp8_decode<256><<<dim3((unsigned)gx, (unsigned)bg), kScF8Warps * 32, smem, st>>>(
            p, (const __nv_bfloat16 *)Q, (const uint8_t *)K8, ksc, LSE, out, out_stride);
    }
    count_launch();
    return cudaGetLastError();
}

bool sparse_fp8_supported(const Params &p, hs2_dtype dt)
{
    auto m8 = [](int64_t x) { return x % 8 == 0; };
    auto m16 = [](int64_t x) { return x % 16 == 0; };
    if (p.ks_t > 0x7fffffffLL) return false;
    return dt == HS2_BF16 && p.D == HD && p.G >= 1 && p.G <= 8 && m8(p.qs_b) && m8(p.qs_t) && m8(p.qs_h) && m16(p.ks_b) &&
           m16(p.ks_t) && m16(p.ks_h) && m8(p.os_b) && m8(p.os_t) && m8(p.os_h);
}

cudaError_t launch_sparse_fp8_prefill(const Params &p, const void *Q, const void *K, const void *V, const float *ksc,
                                      const float *vsc, const int32_t *idx, const float *sink, void *O, float *LSE,
                                      cudaStream_t st)
{
    static bool done[64] = {};
    cudaError_t e = set_smem(k_sparse_fp8_prefill, kPrefillSmem, done);
    if (e != cudaSuccess) return e;
    const int64_t items = (int64_t)p.B * p.Hkv * p.Lq;
    if (items <= 0) return cudaSuccess;
    const int64_t grid = (items + HS2_F8_WARPS - 1) / HS2_F8_WARPS;
    if (grid > 0x7fffffffLL) return cudaErrorNotSupported;
    k_sparse_fp8_prefill<<<(unsigned)grid, HS2_F8_WARPS * 32, kPrefillSmem, st>>>(
        p, (const __nv_bfloat16 *)Q, (const uint8_t *)K, (const uint8_t *)V, ksc, vsc, idx, sink, (__nv_bfloat16 *)O, LSE);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_sparse_fp8_decode(const Params &p, const void *Q, const void *K, const void *V, const float *ksc,
                                     const float *vsc, const int32_t *idx, const float *sink, void *O, float *LSE,
                                     cudaStream_t st, float *raw)
{
    static bool done[64] = {};
    cudaError_t e = set_smem(k_sparse_fp8_decode, kDecodeSmem, done);
    if (e != cudaSuccess) return e;
    const int64_t pairs = (int64_t)p.B * p.Hkv;
    if (pairs <= 0) return cudaSuccess;
    if (pairs > 0x7fffffffLL) return cudaErrorNotSupported;
    k_sparse_fp8_decode<<<(unsigned)pairs, HS2_F8D_WARPS * 32, kDecodeSmem, st>>>(
        p, (const __nv_bfloat16 *)Q, (const uint8_t *)K, (const uint8_t *)V, ksc, vsc, idx, sink, (__nv_bfloat16 *)O, LSE, raw);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hs2
