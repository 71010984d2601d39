// Full causal attention on the 5th-generation tensor cores (tcgen05 + TMEM), bf16, head_dim 128 or 256
// (Section 3.4: the full-attention layer; NoPE, Section 4.1).
//
// One CTA = 128 queries of one head (MMA M = 128), 128 HV + 64 threads (HV = threads per query row, 1 by default),
// two CTAs per SM at head_dim 128 so that one CTA's softmax overlaps the other's tensor work:
//   softmax warps (the first 4 HV warps): HV = 1: one thread per query row; HV = 2: warps w and w+4 share the 32 TMEM
//            lanes of quarter w and take 32 keys of a tile each, the tile maximum agreed through shared memory and a
//            named pair barrier (measured slower than HV = 1: the barrier and the doubled per-tile overhead cost more
//            than the extra warps hide).  tcgen05.ld of the row, causal mask, online softmax in the base-2 domain
//            with a lazily updated row maximum (O in TMEM is rescaled only when the maximum grows by more than 2^8,
//            and only then does a softmax thread wait for P V of the previous tile), P written as bf16 pairs over
//            the scores it came from (tcgen05.st).
//   next warp TMA producer: Q once, then K and V tiles of 64 keys, each into a 2-stage ring of its own.  Every tile
//            is a set of 128-byte-swizzled slices ([rows][64 dims]), the canonical UMMA operand layout.
//   last warp MMA issuer: S = Q K^T (M128 N64 K=D) into one of two S buffers in TMEM, and O += P V
//            (M128 N=D K64, P as the tensor-memory A operand, V as an MN-major B operand) into TMEM.
// TMEM: columns 0-63 / 64-127 the two S buffers (P of a tile in the first 32 columns of its buffer), then the
// O accumulator (fp32, lane = query row).
// Every mbarrier wait is bounded; a wait that runs out sets a bit in a device error word, makes the CTA abandon
// its loops (partners leave together through the predicate of their pair barrier), and the CTA still frees its
// TMEM before it returns.
#include <cuda.h>

#include <type_traits>

#include "hs2_common.cuh"
#include "hs2_tc5.cuh"

namespace hs2 {

__device__ unsigned g_tc5_error;   // bit 0: an mbarrier wait ran out; bit 1: shared-memory base not alignable

namespace {

constexpr int BM = 128, BN = 64, HD = 128;
constexpr uint32_t kBarBytes = 128;
constexpr uint32_t kAlignSlack = 896;             // the dynamic window is at least 128-byte aligned
constexpr uint32_t kTmemCols = 256;               // score kernels, attention at head_dim 128
// shared-memory plan of the attention kernel for head_dim D (a multiple of 64): every operand tile is a set
// of D/64 slices of [rows][64 dims] = 128-byte rows, each slice 128-byte swizzled
template <int D>
struct FaCfg {
    static constexpr int NQ = D / 64;
    static constexpr uint32_t kQBytes = NQ * BM * 128;
    static constexpr uint32_t kKVStage = NQ * BN * 128;       // one K (or V) tile
    static constexpr uint32_t kOffQ = 0;
    static constexpr uint32_t kOffK = kOffQ + kQBytes;        // 2 stages
    static constexpr uint32_t kOffV = kOffK + 2 * kKVStage;   // 2 stages
    static constexpr uint32_t kOffX = kOffV + 2 * kKVStage;   // exchange between the two threads of a row: 6 x 128 floats
    static constexpr uint32_t kOffBar = kOffX + 6 * BM * 4;
    static constexpr uint32_t kSmemBytes = kOffBar + kBarBytes + kAlignSlack;   // 102400 at D=128: two CTAs per SM
    static constexpr uint32_t kTmem = D <= 128 ? 256 : 512;  // 2 x 64 score columns + D output columns, a power of two
    static constexpr int kMinBlocks = D <= 128 ? 2 : 1;
    template <int HV> static constexpr int threads() { return 128 * HV + 64; }   // softmax warps + TMA warp + MMA warp
};
// Threads per query row.  Measured on B200: at head_dim 128 (two CTAs per SM) and at head_dim 256 (one CTA per SM).
#ifndef HS2_FA_HV128
#define HS2_FA_HV128 1
#endif
#ifndef HS2_FA_HV256
#define HS2_FA_HV256 1
#endif
template <int D> struct FaShape { static constexpr int HV = D <= 128 ? HS2_FA_HV128 : HS2_FA_HV256; };
constexpr float kRescaleThreshold = 8.f;          // log2 units

enum Bar { Q_FULL = 0, K_FULL0, K_FULL1, V_FULL0, V_FULL1, S_FULL0, S_FULL1, S_FREE0, S_FREE1, P_FULL0, P_FULL1, PV_DONE0, PV_DONE1, N_BARS };

using namespace tc5;

// bounded wait bound to this file's error word
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    return tc5::mbar_wait(bar, parity, abort_flag, &g_tc5_error);
}

template <int D, int HV>
__global__ void __launch_bounds__(FaCfg<D>::template threads<HV>(), FaCfg<D>::kMinBlocks)
k_full_tc5(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
           const __grid_constant__ CUtensorMap tmV, const Params p, __nv_bfloat16 *__restrict__ O,
           float *__restrict__ LSE, int head_major)
{
    using F = FaCfg<D>;
    constexpr int NQ = F::NQ;
    constexpr uint32_t kQBytes = F::kQBytes, kKVStage = F::kKVStage, kOffQ = F::kOffQ, kOffK = F::kOffK, kOffV = F::kOffV,
                       kOffX = F::kOffX, kOffBar = F::kOffBar, kTmemFa = F::kTmem;
    constexpr int kTmaWarp = 4 * HV, kMmaWarp = 4 * HV + 1;   // behind the softmax warps
    constexpr int EPT = BN / HV;                              // scores per softmax thread and tile
    constexpr int kSoftmaxThreads = 128 * HV;
    extern __shared__ char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    if (pad > kAlignSlack) {   // never seen; refuse rather than run on a misaligned tile
        if (threadIdx.x == 0) atomicOr(&g_tc5_error, 2u);
        return;
    }
    char *smem = smem_raw + pad;
    const uint32_t sbase = raw + pad;
    const uint32_t bars = sbase + kOffBar;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kOffBar + N_BARS * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffBar + N_BARS * 8 + 4);
    auto bar = [&](int i) { return bars + 8u * i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // One-dimensional grid; CTAs start in order of their index.  head_major = 0: (sequence, head) fastest and the query
    // tile descending, so ALL heads' longest tiles run first and the last CTAs to start are the shortest ones.  (With
    // the heads as the slow index every head's long tiles start in turn - on the 8K benchmark the last head's
    // 130-microsecond tile at 460 of 590 microseconds, and SMs finished between 479 and 593.)  head_major = 1: one
    // head after the other, long tiles first within a head: the CTAs in flight then share one KV head, which is worth
    // more than the tail once the cache no longer fits L2 and the kernel runs for a hundred waves.
    const int n_bh = p.B * p.Hq;
    const int n_mblk = (int)(gridDim.x / n_bh);
    const int mblk = n_mblk - 1 - (int)(head_major ? blockIdx.x % n_mblk : blockIdx.x / n_bh);
    const int bh = (int)(head_major ? blockIdx.x / n_mblk : blockIdx.x % n_bh);
    const int h = bh % p.Hq, b = bh / p.Hq;
    const int gkv = h / p.G;
    const int i0 = mblk * BM;
    const int kvl = kvlen_of(p, b);
    const int pos0 = pos_of(p, b, i0);
    const int rows_here = min(BM, p.Lq - i0);
    const int n_vis = max(0, min(pos0 + rows_here, kvl));
    const int nblk = (n_vis + BN - 1) / BN;

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(Q_FULL), 1);
        mbar_init(bar(K_FULL0), 1); mbar_init(bar(K_FULL1), 1);
        mbar_init(bar(V_FULL0), 1); mbar_init(bar(V_FULL1), 1);
        mbar_init(bar(S_FULL0), 1); mbar_init(bar(S_FULL1), 1);
        mbar_init(bar(S_FREE0), kSoftmaxThreads); mbar_init(bar(S_FREE1), kSoftmaxThreads);
        mbar_init(bar(P_FULL0), kSoftmaxThreads); mbar_init(bar(P_FULL1), kSoftmaxThreads);
        mbar_init(bar(PV_DONE0), 1); mbar_init(bar(PV_DONE1), 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == kMmaWarp) {   // TMEM allocation is a warp-wide operation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(kTmemFa) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == kTmaWarp) {
        // ------------------------------------------------ TMA producer
        if (elect_one() && nblk > 0) {
            mbar_expect_tx(bar(Q_FULL), kQBytes);
#pragma unroll
            for (int sl = 0; sl < NQ; ++sl) tma_load_4d(sbase + kOffQ + sl * BM * 128, &tmQ, bar(Q_FULL), 64 * sl, h, i0, b);
            // K and V travel in rings of their own (two stages each).  A K stage is free again as soon as Q K^T of the
            // tile two back has run (the event S_FULL of that tile), a V stage when its P V has (PV_DONE): K runs a whole
            // tile ahead of V, so the next scores are in tensor memory before the softmax asks for them.
            int k_issued = 0, v_issued = 0;
            for (int j = 0; j < nblk; ++j) {
                const int st = j & 1;
                if (j >= 2 && !mbar_wait(bar(S_FULL0 + st), ((j - 2) >> 1) & 1, abort_flag)) break;
                mbar_expect_tx(bar(K_FULL0 + st), kKVStage);
                const uint32_t kdst = sbase + kOffK + st * kKVStage, vdst = sbase + kOffV + st * kKVStage;
#pragma unroll
                for (int sl = 0; sl < NQ; ++sl) tma_load_4d(kdst + sl * BN * 128, &tmK, bar(K_FULL0 + st), 64 * sl, gkv, j * BN, b);
                k_issued = j + 1;
                if (j >= 2 && !mbar_wait(bar(PV_DONE0 + st), ((j - 2) >> 1) & 1, abort_flag)) break;
                mbar_expect_tx(bar(V_FULL0 + st), kKVStage);
#pragma unroll
                for (int sl = 0; sl < NQ; ++sl) tma_load_4d(vdst + sl * BN * 128, &tmV, bar(V_FULL0 + st), 64 * sl, gkv, j * BN, b);
                v_issued = j + 1;
            }
            if (*abort_flag) {   // leaving early: let the copies already in flight land before the CTA goes away
                for (int j = max(0, k_issued - 2); j < k_issued; ++j)
                    for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar(K_FULL0 + (j & 1)), (j >> 1) & 1); ++it) {}
                for (int j = max(0, v_issued - 2); j < v_issued; ++j)
                    for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar(V_FULL0 + (j & 1)), (j >> 1) & 1); ++it) {}
                for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar(Q_FULL), 0); ++it) {}
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------ MMA issuer
        if (elect_one() && nblk > 0) {
            constexpr uint32_t idS = idesc(BM, BN, 0), idPV = idesc(BM, D, 1);
            bool ok = mbar_wait(bar(Q_FULL), 0, abort_flag);
            auto issue_s = [&](int j) -> bool {
                const int st = j & 1, ph = (j >> 1) & 1;
                if (!mbar_wait(bar(K_FULL0 + st), ph, abort_flag)) return false;
                if (!mbar_wait(bar(S_FREE0 + st), ph ^ 1, abort_flag)) return false;
                tc_fence_after();
                const uint32_t qa = sbase + kOffQ, ka = sbase + kOffK + st * kKVStage;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks & 3) * 32;   // 16 dims = 32 bytes inside the swizzled 128-byte row
                    const uint64_t da = smem_desc(qa + (ks >> 2) * (BM * 128) + off, 16, 1024);
                    const uint64_t db = smem_desc(ka + (ks >> 2) * (BN * 128) + off, 16, 1024);
                    umma(tmem + st * BN, da, db, idS, ks > 0);
                }
                umma_commit(bar(S_FULL0 + st));
                return true;
            };
            ok = ok && issue_s(0);
            for (int j = 0; ok && j < nblk; ++j) {
                if (j + 1 < nblk && !issue_s(j + 1)) break;
                const int st = j & 1;
                if (!mbar_wait(bar(V_FULL0 + st), (j >> 1) & 1, abort_flag)) break;
                if (!mbar_wait(bar(P_FULL0 + st), (j >> 1) & 1, abort_flag)) break;
                tc_fence_after();
                const uint32_t va = sbase + kOffV + st * kKVStage;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {   // 16 keys per instruction
                    // P: in tensor memory, over the first 32 columns of the score buffer it was computed from
                    // (16 keys = 8 columns of bf16 pairs); the in-order tensor pipe runs Q K^T of tile j+2, which
                    // overwrites that buffer, after this instruction
                    // V: MN-major, 64-dim halves BN*128 bytes apart (leading offset), 8-key groups 1024 bytes apart
                    const uint64_t db = smem_desc(va + kk * 2048, BN * 128, 1024);
                    umma_ts(tmem + 2 * BN, tmem + st * BN + kk * 8, db, idPV, (j > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bar(PV_DONE0 + st));
            }
        }
    } else {
        // ------------------------------------------------ softmax: HV threads per query row, BN / HV keys of a tile each
        const int quarter = warp & 3, half = HV == 2 ? warp >> 2 : 0;
        const int row = quarter * 32 + lane;       // 0..127, TMEM lane
        const int i = i0 + row;
        const int prow = pos0 + row;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        float *s_mx = reinterpret_cast<float *>(smem + kOffX);   // [tile parity][half][row] raw maximum of the half tile
        float *s_l = s_mx + 4 * BM;                              // [half][row] partial denominators
        const int pair_bar = 1 + quarter;          // named barrier of the two warps that share these 32 rows
        constexpr int OCH = D / 32 / HV;           // 32-column chunks of the O row this thread rescales and stores
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;
        float s[EPT];
        for (int j = 0; j < nblk; ++j) {
            const int sb = j & 1;
            if (ok && !__all_sync(0xffffffffu, mbar_wait(bar(S_FULL0 + sb), (j >> 1) & 1, abort_flag))) ok = false;
            float m_raw = -INFINITY;
            if (ok) {   // this thread's scores into registers; the score buffer is then free for Q K^T of tile j+2
                tc_fence_after();
                if constexpr (EPT == 64) {
                    tmem_ld32(lane_base + sb * BN, *reinterpret_cast<float (*)[32]>(&s[0]));
                    tmem_ld32(lane_base + sb * BN + 32, *reinterpret_cast<float (*)[32]>(&s[32]));
                } else {
                    tmem_ld32(lane_base + sb * BN + half * 32, s);
                }
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(bar(S_FREE0 + sb));
            }
            if (ok) {
                const int j0 = j * BN + half * EPT;
                // raw-score maximum; only tiles that touch the diagonal or the end of the cache pay for masking
                if ((j0 + EPT - 1 > pos0) || (j0 + EPT > kvl)) {
#pragma unroll
                    for (int e = 0; e < EPT; ++e)
                        if (j0 + e > prow || j0 + e >= kvl) s[e] = -INFINITY;
                }
                // four independent chains of 3-input maxima
                float mx0 = s[0], mx1 = s[1], mx2 = s[2], mx3 = s[3];
#pragma unroll
                for (int e = 4; e + 8 <= EPT; e += 8) {
                    mx0 = max3(mx0, s[e], s[e + 4]); mx1 = max3(mx1, s[e + 1], s[e + 5]);
                    mx2 = max3(mx2, s[e + 2], s[e + 6]); mx3 = max3(mx3, s[e + 3], s[e + 7]);
                }
                mx0 = fmaxf(mx0, s[EPT - 4]); mx1 = fmaxf(mx1, s[EPT - 3]); mx2 = fmaxf(mx2, s[EPT - 2]); mx3 = fmaxf(mx3, s[EPT - 1]);
                m_raw = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
            }
            if (HV == 2) {
                // the two halves of a row agree on the tile's maximum (and leave the loop together after a failed wait)
                s_mx[((j & 1) * 2 + half) * BM + row] = m_raw;
                if (!group_all(pair_bar, 64, ok)) { ok = false; break; }
                m_raw = fmaxf(m_raw, s_mx[((j & 1) * 2 + (half ^ 1)) * BM + row]);
            } else if (!ok) {
                break;
            }
            const float m_blk = m_raw * p.scale_log2;                 // the scale is positive
            const bool need = m_blk > m_used + kRescaleThreshold;   // also true for the first finite block
            const float m_new = need ? m_blk : m_used;
            const float corr = need ? exp2f(m_used - m_new) : 1.f;  // 0 when nothing was accumulated yet
            // P of this tile goes to the score buffer it came from, which P V of tile j-2 has left (Q K^T of this tile
            // ran behind it in the tensor pipe), so only a rescale of O has to wait for P V of tile j-1.  One barrier
            // per tile parity: P V of tile j-3 is certainly complete here, so the awaited phase is never ambiguous.
            if (j > 0 && __any_sync(0xffffffffu, need)) {
                if (!__all_sync(0xffffffffu, mbar_wait(bar(PV_DONE0 + ((j - 1) & 1)), ((j - 1) >> 1) & 1, abort_flag))) {
                    ok = false;
                    if (HV == 2) continue;   // the partner learns at the next pair barrier
                    break;
                }
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < OCH; ++c) {   // this thread's columns of the O row (a warp-wide TMEM access)
                    float o[32];
                    const uint32_t oc = lane_base + 2 * BN + (half * OCH + c) * 32;
                    tmem_ld32(oc, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) o[e] *= corr;
                    tmem_st32(oc, o);
                }
                tmem_wait_st();
            }
            l *= corr;
            m_used = m_new;
            const float neg_m = m_used == -INFINITY ? 0.f : -m_used;
            uint32_t pk[EPT / 2];
            float l0 = 0.f, l1 = 0.f;
#pragma unroll
            for (int e = 0; e < EPT; e += 2) {
                const float p0 = exp2f(fmaf(s[e], p.scale_log2, neg_m));       // -inf stays -inf -> 0
                const float p1 = exp2f(fmaf(s[e + 1], p.scale_log2, neg_m));
                l0 += p0; l1 += p1;
                pk[e >> 1] = pack_bf16(p0, p1);
            }
            l += l0 + l1;
            // P replaces the scores it came from
            if constexpr (EPT == 64) tmem_st32u(lane_base + sb * BN, pk);
            else tmem_st16u(lane_base + sb * BN + half * (EPT / 2), pk);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(P_FULL0 + sb));
        }
        // ------------------------------------------------ epilogue
        bool have_o = ok && nblk > 0;
        if (have_o) have_o = __all_sync(0xffffffffu, mbar_wait(bar(PV_DONE0 + ((nblk - 1) & 1)), ((nblk - 1) >> 1) & 1, abort_flag));
        if (HV == 2) {
            s_l[half * BM + row] = l;
            have_o = group_all(pair_bar, 64, have_o);
            l += s_l[(half ^ 1) * BM + row];
        }
        tc_fence_after();
        const float inv = l > 0.f ? 1.f / l : 0.f;
        __nv_bfloat16 *orow = O + b * p.os_b + (int64_t)i * p.os_t + h * p.os_h + half * (D / HV);
#pragma unroll
        for (int c = 0; c < OCH; ++c) {
            float o[32];
            if (have_o) {   // uniform across the warp
                tmem_ld32(lane_base + 2 * BN + (half * OCH + c) * 32, o);
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) o[e] = 0.f;
            }
            if (i < p.Lq) {
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint4 v;
                    v.x = pack_bf16(o[8 * q4 + 0] * inv, o[8 * q4 + 1] * inv);
                    v.y = pack_bf16(o[8 * q4 + 2] * inv, o[8 * q4 + 3] * inv);
                    v.z = pack_bf16(o[8 * q4 + 4] * inv, o[8 * q4 + 5] * inv);
                    v.w = pack_bf16(o[8 * q4 + 6] * inv, o[8 * q4 + 7] * inv);
                    *reinterpret_cast<uint4 *>(orow + c * 32 + q4 * 8) = v;
                }
            }
        }
        if (half == 0 && i < p.Lq)
            LSE[((int64_t)b * p.Hq + h) * p.Lq + i] = (have_o && l > 0.f) ? (m_used + log2f(l)) * kLn2 : -INFINITY;
    }
    // ------------------------------------------------ teardown: everybody arrives, then TMEM is returned
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemFa) : "memory");
    }
}


// ---------------------------------------------------------------- selection scores on tcgen05
// a[i][j] = max over the heads h of the group of (scale <q_h(i), k_j> - LSE_h(i))   (Section 3.4)
// One CTA = TQ = NC/G consecutive queries of one (sequence, KV head) x one chunk of keys.  The MMA
// computes S^T = K Q^T: 128 keys on M (TMEM lane = key), the TQ x G (query, head) pairs on N = NC columns,
// so the G heads of a query are adjacent TMEM columns of one lane and their maximum is thread local.
// The subtraction of LSE is one more K step of the same MMA (a key operand of ones against -LSE / scale split into
// three bf16 terms), so the accumulator holds (score / scale) of every (key, query, head).  One warp feeds K tiles by
// TMA (a ring of 2 or 3 stages), one thread issues the MMAs into two accumulator buffers, NC / 16 epilogue warps
// (thread = key; the warps that share the 32 TMEM lanes of a quarter take 64 columns each) take the group maximum and,
// by mode, write 32 consecutive keys of a strip row per warp instruction or append the scores that pass the query's
// threshold to its candidate list.  The epilogue is a chain of TMEM loads and short dependent arithmetic: eight warps
// per 128 columns hide its latency where four left the tensor pipe waiting for a free accumulator.
#ifndef HS2_SC_KSTAGES
#define HS2_SC_KSTAGES 3   // key tiles in flight in a 256-column CTA (2 to 5); measured on the 128K layer: 2: 221 ms, 3: 219 ms, 4: 237 ms
#endif
#ifndef HS2_SC_WIDE
#define HS2_SC_WIDE 1   // 256-column CTAs of the score sweep for head_dim 128 and groups of 8 or 16 (0: 128 columns everywhere)
#endif
#ifndef HS2_SC_KCHUNK
#define HS2_SC_KCHUNK 4096
#endif
constexpr int SC_KCHUNK = HS2_SC_KCHUNK;                  // keys per CTA
// NC = 128 columns: 8 epilogue warps, two CTAs per SM (tensor memory: 2 x 2 x 128 columns).  NC = 256 (head_dim 128):
// 16 epilogue warps, one CTA per SM with all of tensor memory.  An M128 N128 K16 instruction reads 8 KB of operands in
// the 64 cycles it takes - the whole bandwidth of shared memory, which the TMA writes of the key tiles want too; at
// N = 256 it is 12 KB per 128 cycles, and a key tile is loaded once per 256 columns instead of once per 128.
// shared-memory plan of the score sweep for head_dim D: Q and K tiles are D/64 slices of [128 rows][128 B]
template <int D, int NC = 128>
struct ScCfg {
    static constexpr int NQ = D / 64;
    static constexpr int kTmaWarp = NC / 16, kMmaWarp = NC / 16 + 1;   // after the (up to) NC / 16 epilogue warps
    static constexpr int kThreads = (NC / 16 + 2) * 32;
    static constexpr uint32_t kTmem = 2 * NC;                     // two accumulator buffers
    static constexpr uint32_t kSlice = 128 * 128;                 // one slice of a key tile: 128 rows of 128 bytes
    static constexpr uint32_t kSliceQ = NC * 128;                 // one slice of the (query, head) rows
    static constexpr uint32_t kOffQ = 0;                          // (query, head) rows
    static constexpr int KS = NC == 256 ? HS2_SC_KSTAGES : 2;     // depth of the ring of key tiles
    static constexpr uint32_t kOffK = NQ * kSliceQ;               // KS stages of key rows
    static constexpr uint32_t kOffAug = kOffK + KS * NQ * kSlice; // one extra K step: [128][16] and [NC][16] bf16, 32-byte swizzle
    static constexpr uint32_t kOffNl = kOffAug + 4096 + NC * 32;  // float[NC]: -LSE/scale per column
    static constexpr uint32_t kOffNq = kOffNl + NC * 4;           // int[NC]: keys needed per query
    static constexpr uint32_t kOffRow = kOffNq + NC * 4;          // int64[NC]: strip row of each query
    static constexpr uint32_t kOffTau = kOffRow + NC * 8;         // uint32[32]: filter threshold per query (filter mode)
    static constexpr uint32_t kOffCnt = kOffTau + 128;            // int[32]: candidates appended per query (filter mode)
    static constexpr uint32_t kOffBar = kOffCnt + 1024;
    static constexpr uint32_t kSmemBytes = kOffBar + kBarBytes + kAlignSlack;
    static constexpr int kMinBlocks = (D <= 128 && NC == 128) ? 2 : 1;
    // (the 18 warps of NC = 256 get 96 registers per thread: the register file is handed out as if a CTA had a multiple
    // of four warps, and a launch that asks for 112 is refused)
    static_assert(kSmemBytes <= 227 * 1024, "fits the shared memory of one SM");
};
// the key ring has up to five stages (SK_FULL0 + s, SK_EMPTY0 + s); the accumulator is double-buffered
enum ScBar { SQ_FULL = 0, ACC_FULL0, ACC_FULL1, ACC_FREE0, ACC_FREE1, SK_FULL0 = 5, SK_EMPTY0 = 10, SC_N_BARS = 15 };

// What the sweep does with a score:
//   SC_STRIP   write it to the strip row at its key position (keys split into chunks over blockIdx.x)
//   SC_SAMPLE  only every `samp`-th key tile is computed; written compactly (tile t of the sample at 128 t)
//   SC_FILTER  one CTA sweeps all keys of its queries and appends (score, key) of every score whose order key
//              is >= the query's threshold to that query's candidate list (in no particular order).  A list is four
//              sub-lists, one per quarter of a key tile (keys 32 q .. 32 q + 31 of every 128): the one warp that
//              owns a (query, quarter) counts its sub-list in a register, so appending needs no atomic
enum { SC_STRIP = 0, SC_SAMPLE = 1, SC_FILTER = 2 };

struct FilterBuf {
    const uint32_t *tau_key;   // [rows of the block] threshold as order-preserving key
    int2 *cand;                // [rows][4][cap / 4] records: x = bits of score / scale (the accumulator's value), y = the key
    int *count;                // [rows][4] candidates found per sub-list (may exceed cap / 4: then the row is redone elsewhere; -1: gave up)
    int cap;                   // multiple of 4
};

// the float whose order key is `key`; the two sentinels of the filter thresholds map to values that make the
// comparison `score >= threshold` come out right: key 0 (every score passes) -> -inf, key 0xffffffff (none) -> NaN
__device__ __forceinline__ float key_to_float(uint32_t key)
{
    if (key == 0u) return -INFINITY;
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

template <int G, int MODE, int D, int NC>
__global__ void __launch_bounds__(ScCfg<D, NC>::kThreads, ScCfg<D, NC>::kMinBlocks)
k_scores_tc5(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const Params p,
             const float *__restrict__ LSE, float *__restrict__ out, int64_t out_stride, int64_t row0, int64_t n_rows,
             int all_visible, int tile_first, int tiles_per_bg, int samp, FilterBuf fb)
{
    using S = ScCfg<D, NC>;
    constexpr int kScTmaWarp = S::kTmaWarp, kScMmaWarp = S::kMmaWarp;
    constexpr int NQ = S::NQ, KS = S::KS;
    constexpr uint32_t kScOffQ = S::kOffQ, kScOffK = S::kOffK, kScOffNl = S::kOffNl, kScOffNq = S::kOffNq,
                       kScOffRow = S::kOffRow, kScOffTau = S::kOffTau, kScOffCnt = S::kOffCnt, kScOffBar = S::kOffBar,
                       kStage = NQ * S::kSlice, kStageQ = NQ * S::kSliceQ;
    constexpr int TQ = NC / G;                     // queries per CTA
    constexpr int QPC = G <= 32 ? 32 / G : 1;      // queries per 32-column chunk when a group fits a chunk
    constexpr int CPQ = G <= 32 ? 1 : G / 32;      // 32-column chunks per query otherwise
    constexpr int EW = NC / (G <= 64 ? 64 : G);    // epilogue warps per TMEM lane quarter (a query's columns stay in one warp)
    constexpr int CPW = NC / 32 / EW;              // 32-column chunks per epilogue warp
    constexpr int TQW = TQ / EW;                   // queries per epilogue warp
    constexpr int kEpiThreads = 128 * EW;
    static_assert(NC % G == 0 && (G <= 32 || G % 32 == 0), "the group's heads tile the columns");
    static_assert(MODE != SC_FILTER || TQ <= 32, "filter mode keeps one pass bit per query");
    extern __shared__ char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    if (pad > kAlignSlack) {
        if (threadIdx.x == 0) atomicOr(&g_tc5_error, 2u);
        return;
    }
    char *smem = smem_raw + pad;
    const uint32_t sbase = raw + pad;
    const uint32_t bars = sbase + kScOffBar;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kScOffBar + SC_N_BARS * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kScOffBar + SC_N_BARS * 8 + 4);
    auto bar = [&](int i) { return bars + 8u * i; };
    float *s_nl = reinterpret_cast<float *>(smem + kScOffNl);
    int *s_nq = reinterpret_cast<int *>(smem + kScOffNq);
    int64_t *s_row = reinterpret_cast<int64_t *>(smem + kScOffRow);
    uint32_t *s_tau = reinterpret_cast<uint32_t *>(smem + kScOffTau);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // flattened (b, g, query tile); the filter sweep walks all keys per CTA, so its long tiles (late queries) go first
    const int tile = tile_first + (MODE == SC_FILTER ? (int)(gridDim.y - 1 - blockIdx.y) : (int)blockIdx.y);
    const int bg = tile / tiles_per_bg;
    const int qt = tile % tiles_per_bg;
    const int gkv = bg % p.Hkv, b = bg / p.Hkv;
    const int kvl = kvlen_of(p, b);
    const int iq0 = qt * TQ;
    const int64_t bg_row0 = (int64_t)bg * p.Lq;
    const int i_lo = (int)max((int64_t)0, row0 - bg_row0), i_hi = (int)min((int64_t)p.Lq, row0 + n_rows - bg_row0);
    const int c_lo = max(iq0, i_lo), c_hi = min(iq0 + TQ, i_hi);
    if (c_lo >= c_hi) return;
    auto n_of = [&](int i) {
        const int pos = pos_of(p, b, i);
        return max(0, min(all_visible ? pos + 1 : pos - p.w + 1, kvl));
    };
    const int limit = n_of(c_hi - 1);
    // key tiles of this CTA: tile t of the loop is key tile (kt0 + t) * kstep
    const int kstep = MODE == SC_SAMPLE ? samp : 1;
    const int kt0 = MODE == SC_FILTER ? 0 : blockIdx.x * (SC_KCHUNK / 128);
    const int tiles_total = (limit + 128 * kstep - 1) / (128 * kstep);   // key tiles (of this stride) that start below the limit
    const int ntile = MODE == SC_FILTER ? tiles_total : min(SC_KCHUNK / 128, tiles_total - kt0);
    if (MODE == SC_FILTER) {
        if (blockIdx.x != 0) return;
        if (ntile <= 0) {   // no candidates at all: the lists are empty
            if (tid < 4 * TQ && iq0 + tid / 4 >= c_lo && iq0 + tid / 4 < c_hi) fb.count[(bg_row0 + iq0 + tid / 4 - row0) * 4 + (tid & 3)] = 0;
            return;
        }
    } else if (ntile <= 0) {
        return;
    }

    if (tid < NC) {   // per-column constants
        const int t = tid / G, hh = tid % G;
        const int i = iq0 + t;
        const bool ok = i >= c_lo && i < c_hi;
        // G is the group size rounded up to a tile-able one; columns past the real group hold some other head's
        // (or zero-filled) scores and are taken out of the maximum by -inf
        const float nl = !ok ? 0.f : hh < p.G ? -LSE[((int64_t)b * p.Hq + gkv * p.G + hh) * p.Lq + i] / p.scale : -INFINITY;
        s_nl[tid] = nl;
        // The subtraction of LSE rides on the tensor cores: one more K step whose key operand is all ones and whose
        // (query, head) operand holds nl as three bf16 terms (hi + mid + lo carry 24 bits), the other 13 entries zero.
        // Only the sum over a row's 16 entries matters, so the order of the two 16-byte chunks inside a row is free.
        const bool fin = fabsf(nl) <= 3.0e38f;
        const __nv_bfloat16 hi = __float2bfloat16_rn(nl);
        const float r1 = fin ? nl - __bfloat162float(hi) : 0.f;
        const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
        const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
        uint4 c0;
        c0.x = (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(mid) << 16);
        c0.y = (uint32_t)__bfloat16_as_ushort(lo);
        c0.z = 0u; c0.w = 0u;
        uint4 *qaug = reinterpret_cast<uint4 *>(smem + S::kOffAug + 4096 + tid * 32);
        qaug[0] = c0;
        qaug[1] = make_uint4(0u, 0u, 0u, 0u);
        if (hh == 0) {
            s_nq[t] = ok ? n_of(i) : 0;
            s_row[t] = ok ? (bg_row0 + i - row0) : -1;
            if (MODE == SC_FILTER && t < 32) {
                s_tau[t] = ok ? fb.tau_key[bg_row0 + i - row0] : 0xffffffffu;
            }
        }
    }
    if (tid < 256)   // the all-ones key operand of the extra step (128 rows of 32 bytes)
        reinterpret_cast<uint4 *>(smem + S::kOffAug)[tid] = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u);
    fence_proxy_async();   // the tensor cores read what these threads wrote
    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(SQ_FULL), 1);
        for (int s = 0; s < KS; ++s) { mbar_init(bar(SK_FULL0 + s), 1); mbar_init(bar(SK_EMPTY0 + s), 1); }
        mbar_init(bar(ACC_FULL0), 1); mbar_init(bar(ACC_FULL1), 1);
        mbar_init(bar(ACC_FREE0), kEpiThreads); mbar_init(bar(ACC_FREE1), kEpiThreads);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == kScMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(S::kTmem) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == kScTmaWarp) {
        if (elect_one()) {
            mbar_expect_tx(bar(SQ_FULL), kStageQ);
#pragma unroll
            for (int sl = 0; sl < NQ; ++sl) tma_load_4d(sbase + kScOffQ + sl * S::kSliceQ, &tmQ, bar(SQ_FULL), 64 * sl, gkv * p.G, iq0, b);
            int issued = 0;
            for (int t = 0; t < ntile; ++t) {
                const int st = t % KS;
                if (!mbar_wait(bar(SK_EMPTY0 + st), ((t / KS) & 1) ^ 1, abort_flag)) break;
                issued = t + 1;
                mbar_expect_tx(bar(SK_FULL0 + st), kStage);
                const uint32_t kdst = sbase + kScOffK + st * kStage;
                const int krow = (kt0 + t) * kstep * 128;
#pragma unroll
                for (int sl = 0; sl < NQ; ++sl) tma_load_4d(kdst + sl * S::kSlice, &tmK, bar(SK_FULL0 + st), 64 * sl, gkv, krow, b);
            }
            if (*abort_flag) {
                for (int t = max(0, issued - KS); t < issued; ++t)
                    for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar(SK_FULL0 + t % KS), (t / KS) & 1); ++it) {}
                for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar(SQ_FULL), 0); ++it) {}
            }
        }
    } else if (warp == kScMmaWarp) {
        if (elect_one()) {
            constexpr uint32_t id = idesc(128, NC, 0);
            bool ok = mbar_wait(bar(SQ_FULL), 0, abort_flag);
            for (int t = 0; ok && t < ntile; ++t) {
                const int st = t % KS, ab = t & 1;
                if (!mbar_wait(bar(SK_FULL0 + st), (t / KS) & 1, abort_flag)) break;
                if (!mbar_wait(bar(ACC_FREE0 + ab), ((t >> 1) & 1) ^ 1, abort_flag)) break;
                tc_fence_after();
                const uint32_t ka = sbase + kScOffK + st * kStage, qa = sbase + kScOffQ;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks >> 2) * S::kSlice + (ks & 3) * 32, offq = (ks >> 2) * S::kSliceQ + (ks & 3) * 32;
                    umma(tmem + ab * NC, smem_desc(ka + off, 16, 1024), smem_desc(qa + offq, 16, 1024), id, ks > 0);
                }
                umma(tmem + ab * NC, smem_desc_sw32(sbase + S::kOffAug, 256), smem_desc_sw32(sbase + S::kOffAug + 4096, 256), id, 1);   // - LSE / scale
                umma_commit(bar(SK_EMPTY0 + st));
                umma_commit(bar(ACC_FULL0 + ab));
            }
        }
    } else if (warp < 4 * EW) {
        const int quarter = warp & 3, half = warp >> 2;
        const int row = quarter * 32 + lane;   // key inside the tile = TMEM lane
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        const int q_first = half * TQW;        // this warp's queries: q_first .. q_first + TQW - 1
        const unsigned lt_mask = (1u << lane) - 1u;
        // per-query constants in registers when a warp owns few queries (they are read once per score otherwise)
        constexpr bool kHoist = TQW <= 8;
        int nq_r[kHoist ? TQW : 1];
        float *orow_r[kHoist && MODE != SC_FILTER ? TQW : 1];
        float tau_r[kHoist && MODE == SC_FILTER ? TQW : 1];   // thresholds in the accumulator's units: one compare per score
        int rb_r[kHoist && MODE == SC_FILTER ? TQW : 1];      // first slot of this warp's sub-list of the query's candidates (the lists of a block hold < 2^28 entries)
        int cnt_r[MODE == SC_FILTER ? TQW : 1];               // entries this warp has appended per query (warp-uniform)
        const int capq = MODE == SC_FILTER ? fb.cap >> 2 : 0;
        // The filter compares the accumulator (score / scale) with threshold / scale, lowered by a few units in the
        // last place: every score that reaches the threshold after the multiplication by scale passes (the list may
        // hold a few more, which is harmless: the select works on the stored scores), and the multiplication is
        // paid by the few scores that pass, not by all.
        auto raw_tau = [&](uint32_t tk) {
            const float t = key_to_float(tk) / p.scale;   // -inf stays -inf (all pass), NaN stays NaN (none)
            return t - fabsf(t) * 4.8e-7f - 1e-30f;
        };
        int nq_min = 0x7fffffff;   // tiles that end below it need no causal test in this warp
        if (MODE == SC_FILTER) {
#pragma unroll
            for (int q = 0; q < TQW; ++q) {
                cnt_r[q] = 0;
                nq_min = min(nq_min, s_nq[q_first + q]);
            }
        }
        if (kHoist) {
#pragma unroll
            for (int q = 0; q < TQW; ++q) {
                nq_r[q] = s_nq[q_first + q];
                if (MODE != SC_FILTER) orow_r[q] = out + s_row[q_first + q] * out_stride;   // never used when nq is 0
                if (MODE == SC_FILTER) {
                    tau_r[q] = raw_tau(s_tau[q_first + q]);
                    rb_r[q] = (int)(s_row[q_first + q] * fb.cap) + quarter * capq;
                }
            }
        }
        bool alive = true;
        bool room = false;       // every sub-list of this warp can take a whole tile's worth of entries
        int t_recheck = 0;       // the tile at which that has to be looked at again
        const unsigned lane_bit = 1u << lane;
        // one key tile: CHECK = false when every key of the tile is visible to every query of this warp
        auto do_tile = [&](int t, auto check_tag) {
            constexpr bool CHECK = decltype(check_tag)::value;
            const int ab = t & 1;
            const int key = (kt0 + t) * kstep * 128 + row;
            const int col = MODE == SC_SAMPLE ? (kt0 + t) * 128 + row : key;
            float aval[MODE == SC_FILTER ? TQW : 1];      // accumulator maxima (score / scale)
            unsigned mq[MODE == SC_FILTER ? TQW : 1];     // per query: the lanes whose score passes the filter
            float carry = -INFINITY;   // running group maximum when a group spans several chunks
#pragma unroll
            for (int c = 0; c < CPW; ++c) {
                const int cc = half * CPW + c;   // 32-column chunk of the accumulator
                float v[32];
                tmem_ld32(lane_base + ab * NC + cc * 32, v);
                tmem_wait_ld();
                if (c == CPW - 1) {   // the last chunk is in registers: the accumulator goes back to the tensor core
                    tc_fence_before();   // before the arithmetic on it, not after
                    mbar_arrive(bar(ACC_FREE0 + ab));
                }
#pragma unroll
                for (int q = 0; q < QPC; ++q) {
                    constexpr int W = G <= 32 ? G : 32;   // columns of this chunk that belong to one query
                    float a = v[q * W];
#pragma unroll
                    for (int hh = 1; hh + 1 < W; hh += 2) a = max3(a, v[q * W + hh], v[q * W + hh + 1]);
                    if (W % 2 == 0 && W > 1) a = fmaxf(a, v[q * W + W - 1]);
                    if (CPQ > 1) {
                        carry = fmaxf(carry, a);
                        if ((c + 1) % CPQ != 0) continue;   // more chunks of this query follow
                        a = carry;
                        carry = -INFINITY;
                    }
                    const int ql = CPQ > 1 ? c / CPQ : c * QPC + q;   // query inside this warp's set
                    const int tq = q_first + ql;
                    if (MODE == SC_FILTER) {
                        aval[ql] = a;
                        // (float order and key order agree: -0 and +0 are one key, NaN scores are a caller error)
                        const float tau = kHoist ? tau_r[kHoist ? ql : 0] : raw_tau(s_tau[tq]);
                        bool pass = a >= tau;
                        if (CHECK) pass = pass && key < (kHoist ? nq_r[kHoist ? ql : 0] : s_nq[tq]);
                        mq[ql] = __ballot_sync(0xffffffffu, pass);
                    } else if (key < (kHoist ? nq_r[kHoist ? ql : 0] : s_nq[tq])) {
                        const float av = a * p.scale;
                        if (kHoist) orow_r[kHoist ? ql : 0][col] = av;
                        else out[s_row[tq] * out_stride + col] = av;
                    }
                }
            }
            if (MODE == SC_FILTER) {
                // Append in no particular order.  This warp is the only writer of its sub-list of every query it owns,
                // so the fill counts live in registers (the same in every lane): the ballot taken at the compare gives
                // every passing lane its rank, then one store.  The queries are independent of one another - no
                // atomic, no shared memory, no dependent chain from one query to the next (an atomic per (query, warp,
                // tile) on a shared counter plus a shuffle of its result made the appends one long latency chain).
                // A tile adds at most 32 entries to a sub-list, so the test against the capacity is made per tile,
                // and only once the fullest sub-list could reach it (never, for a list that stays inside its six
                // standard deviations); until then no append looks at the capacity.
                if (t >= t_recheck) {
                    int cmax = cnt_r[0];
#pragma unroll
                    for (int q = 1; q < TQW; ++q) cmax = max(cmax, cnt_r[q]);
                    room = cmax + 32 <= capq;
                    t_recheck = room ? t + (capq - cmax) / 32 : t + 1;
                }
                auto append = [&](auto room_tag) {
                    constexpr bool ROOM = decltype(room_tag)::value;
#pragma unroll
                    for (int q = 0; q < TQW; ++q) {
                        const unsigned m = mq[q];
                        const int pos = cnt_r[q] + __popc(m & lt_mask);
                        if ((m & lane_bit) && (ROOM || pos < capq)) {
                            const int64_t o = kHoist ? (int64_t)(rb_r[kHoist ? q : 0] + pos)
                                                     : s_row[q_first + q] * fb.cap + quarter * capq + pos;
                            fb.cand[o] = make_int2(__float_as_int(aval[q]), key);   // one 8-byte store; the select scales the score
                        }
                        cnt_r[q] += __popc(m);
                    }
                };
                if (room) append(std::true_type{});
                else append(std::false_type{});
            }
        };
        for (int t = 0; t < ntile; ++t) {
            if (!__all_sync(0xffffffffu, mbar_wait(bar(ACC_FULL0 + (t & 1)), (t >> 1) & 1, abort_flag))) { alive = false; break; }
            tc_fence_after();
            if (MODE == SC_FILTER && (kt0 + t + 1) * kstep * 128 <= nq_min) do_tile(t, std::false_type{});
            else do_tile(t, std::true_type{});
        }
        if (MODE == SC_FILTER) {
            const bool fine = alive && !*abort_flag;   // otherwise the sweep gave up: -1 sends the row to the exact redo
#pragma unroll
            for (int q = 0; q < TQW; ++q)
                if (lane == (q & 31) && s_row[q_first + q] >= 0) fb.count[s_row[q_first + q] * 4 + quarter] = fine ? cnt_r[q] : -1;
        }
    }
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == kScMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(S::kTmem) : "memory");
    }
}

__global__ void k_fill_tc5(float *__restrict__ out, int64_t n, float v)
{
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) out[e] = v;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
bool g_encode_tried = false;

EncodeTiledFn encode_fn()
{
    if (!g_encode_tried) {
        g_encode_tried = true;
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            g_encode = (EncodeTiledFn)fn;
        (void)cudaGetLastError();
    }
    return g_encode;
}

// [B, L, H, 128] bf16 with element strides (sb, st, sh): box = 64 dims x `rows` tokens of one head, 128-byte swizzle
bool make_map(CUtensorMap *tm, const void *base, int B, int L, int H, int64_t sb, int64_t st, int64_t sh, int rows,
              int box_heads = 1, int D = HD)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)L, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)sh * 2, (cuuint64_t)st * 2, (cuuint64_t)sb * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)box_heads, (cuuint32_t)rows, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

namespace tc5 {
bool make_tile_map(CUtensorMap *tm, const void *base, int B, int L, int H, int64_t sb, int64_t st, int64_t sh, int rows,
                   int box_heads, int D)
{
    return make_map(tm, base, B, L, H, sb, st, sh, rows, box_heads, D);
}
bool tma_available() { return encode_fn() != nullptr; }
}  // namespace tc5

bool full_tc5_supported(const Params &p, hs2_dtype dt)
{
    auto m8 = [](int64_t x) { return x % 8 == 0 && x > 0; };
    return dt == HS2_BF16 && p.D == HD && m8(p.qs_b) && m8(p.qs_t) && m8(p.qs_h) && m8(p.ks_b) && m8(p.ks_t) &&
           m8(p.ks_h) && m8(p.os_b) && m8(p.os_t) && m8(p.os_h) && (int64_t)p.B * p.Hq <= 65535 && encode_fn() != nullptr;
}

// the attention kernel alone also covers head_dim 256 (the paper's own model shape, Table 1)
bool full_attn_tc5_supported(const Params &p, hs2_dtype dt)
{
    if (p.D == HD) return full_tc5_supported(p, dt);
    auto m8 = [](int64_t x) { return x % 8 == 0 && x > 0; };
    return dt == HS2_BF16 && p.D == 256 && m8(p.qs_b) && m8(p.qs_t) && m8(p.qs_h) && m8(p.ks_b) && m8(p.ks_t) &&
           m8(p.ks_h) && m8(p.os_b) && m8(p.os_t) && m8(p.os_h) && (int64_t)p.B * p.Hq <= 65535 && encode_fn() != nullptr;
}

template <int D>
cudaError_t launch_fa(const Params &p, const void *Q, const void *K, const void *V, void *O, float *LSE, cudaStream_t st)
{
    CUtensorMap tmQ, tmK, tmV;
    if (!make_map(&tmQ, Q, p.B, p.Lq, p.Hq, p.qs_b, p.qs_t, p.qs_h, BM, 1, D) ||
        !make_map(&tmK, K, p.B, p.Lk, p.Hkv, p.ks_b, p.ks_t, p.ks_h, BN, 1, D) ||
        !make_map(&tmV, V, p.B, p.Lk, p.Hkv, p.ks_b, p.ks_t, p.ks_h, BN, 1, D))
        return cudaErrorNotSupported;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!(dev >= 0 && dev < 64 && attr_set[dev])) {
        if ((e = cudaFuncSetAttribute(k_full_tc5<D, FaShape<D>::HV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FaCfg<D>::kSmemBytes)) != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    dim3 grid((unsigned)(((p.Lq + BM - 1) / BM) * (p.B * p.Hq)));
    // the whole cache of the call against the L2 (126 MB on B200; the test is a fixed 96 MB so that it is the same everywhere)
    const int64_t kv_bytes = (int64_t)p.B * p.Hkv * p.Lk * D * 2 * 2;
    const int head_major = kv_bytes > ((int64_t)96 << 20) ? 1 : 0;
    k_full_tc5<D, FaShape<D>::HV><<<grid, FaCfg<D>::template threads<FaShape<D>::HV>(), FaCfg<D>::kSmemBytes, st>>>(tmQ, tmK, tmV, p, (__nv_bfloat16 *)O, LSE, head_major);
    count_launch();
    return cudaGetLastError();
}

// Returns cudaErrorNotSupported when the tensor maps cannot be built (the caller then takes the mma.sync kernel).
cudaError_t launch_full_attn_tc5(const Params &p, const void *Q, const void *K, const void *V, void *O, float *LSE,
                                 cudaStream_t st)
{
    if (p.D == 128) return launch_fa<128>(p, Q, K, V, O, LSE, st);
    if (p.D == 256) return launch_fa<256>(p, Q, K, V, O, LSE, st);
    return cudaErrorNotSupported;
}

template <int G, int MODE, int D, int NC = 128>
cudaError_t launch_sc(const CUtensorMap &tmQ, const CUtensorMap &tmK, const Params &p, const float *LSE, float *out,
                      int64_t out_stride, int64_t row0, int64_t n_rows, bool all_visible, int samp, const FilterBuf &fb,
                      cudaStream_t st)
{
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!(dev >= 0 && dev < 64 && attr_set[dev])) {
        if ((e = cudaFuncSetAttribute(k_scores_tc5<G, MODE, D, NC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ScCfg<D, NC>::kSmemBytes)) != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    constexpr int TQ = NC / G;
    const int tiles_per_bg = (p.Lq + TQ - 1) / TQ;
    // only the query tiles that intersect rows [row0, row0 + n_rows) of the flattened (b, g, i) index
    const int64_t last = row0 + n_rows - 1;
    const int64_t t_first = (row0 / p.Lq) * tiles_per_bg + (row0 % p.Lq) / TQ;
    const int64_t t_last = (last / p.Lq) * tiles_per_bg + (last % p.Lq) / TQ;
    const int64_t gy = t_last - t_first + 1;
    if (gy > 65535 || t_last > 0x7fffffffLL) return cudaErrorNotSupported;
    const int key_tiles = (p.Lk + 128 * samp - 1) / (128 * samp);
    const unsigned gx = MODE == SC_FILTER ? 1u : (unsigned)((key_tiles + SC_KCHUNK / 128 - 1) / (SC_KCHUNK / 128));
    dim3 grid(gx, (unsigned)gy);
    k_scores_tc5<G, MODE, D, NC><<<grid, ScCfg<D, NC>::kThreads, ScCfg<D, NC>::kSmemBytes, st>>>(tmQ, tmK, p, LSE, out, out_stride, row0, n_rows, all_visible ? 1 : 0,
                                                               (int)t_first, tiles_per_bg, samp, fb);
    count_launch();
    return cudaGetLastError();
}

// smallest instantiated group size >= g (powers of two up to 128), 0 if there is none
int padded_group(int g, int D)
{
    if (D != 128 && D != 256) return 0;
    for (int c = 1; c <= 128; c *= 2)
        if (c >= g) return c;
    return 0;
}

template <int MODE>
cudaError_t launch_sc_mode(const Params &p, const void *Q, const void *K, const float *LSE, float *out, int64_t out_stride,
                           int64_t row0, int64_t n_rows, bool all_visible, int samp, const FilterBuf &fb, cudaStream_t st)
{
    if (n_rows == 0) return cudaSuccess;
    CUtensorMap tmQ, tmK;
    // the kernel is instantiated for groups that tile its 128 columns; any other size runs as the next one up
    // with the surplus columns masked (the sampled and filtered sweeps exist for exact sizes only)
    const int gp = padded_group(p.G, p.D);
    if (gp == 0 || (gp != p.G && MODE != SC_STRIP)) return cudaErrorNotSupported;
    // head_dim 128, groups of 8 and 16: 256 (query, head) columns per CTA (see ScCfg); everything else 128
    const bool wide = HS2_SC_WIDE && p.D == 128 && (gp == 8 || gp == 16);
    const int ncol = wide ? 256 : 128;
    if (!make_map(&tmQ, Q, p.B, p.Lq, p.Hq, p.qs_b, p.qs_t, p.qs_h, ncol / gp, gp, p.D) ||
        !make_map(&tmK, K, p.B, p.Lk, p.Hkv, p.ks_b, p.ks_t, p.ks_h, 128, 1, p.D))
        return cudaErrorNotSupported;
    if ((n_rows + p.Lq) / (ncol / gp) + 2 * (int64_t)p.B * p.Hkv > 65535) return cudaErrorNotSupported;   // grid.y bound
    constexpr int M2 = MODE == SC_FILTER ? SC_STRIP : MODE;   // groups of 1 or 2 have no filter instantiation
    constexpr int M3 = SC_STRIP;                              // large groups and head_dim 256: strips only
#define HS2_SC(G_, MODE_, D_) return launch_sc<G_, MODE_, D_>(tmQ, tmK, p, LSE, out, out_stride, row0, n_rows, all_visible, samp, fb, st)
#if HS2_SC_WIDE
    if (wide) {
        if (gp == 8) return launch_sc<8, MODE, 128, 256>(tmQ, tmK, p, LSE, out, out_stride, row0, n_rows, all_visible, samp, fb, st);
        return launch_sc<16, MODE, 128, 256>(tmQ, tmK, p, LSE, out, out_stride, row0, n_rows, all_visible, samp, fb, st);
    }
#endif
    if (p.D == 128) {
        switch (gp) {
            case 1: if (MODE == SC_FILTER) return cudaErrorNotSupported; HS2_SC(1, M2, 128);
            case 2: if (MODE == SC_FILTER) return cudaErrorNotSupported; HS2_SC(2, M2, 128);
            case 4: HS2_SC(4, MODE, 128);
            case 8: HS2_SC(8, MODE, 128);
            case 16: HS2_SC(16, MODE, 128);
            case 32: if (MODE != SC_STRIP) return cudaErrorNotSupported; HS2_SC(32, M3, 128);
            case 64: if (MODE != SC_STRIP) return cudaErrorNotSupported; HS2_SC(64, M3, 128);
            case 128: if (MODE != SC_STRIP) return cudaErrorNotSupported; HS2_SC(128, M3, 128);
        }
    } else if (p.D == 256) {
        if (MODE != SC_STRIP) return cudaErrorNotSupported;
        switch (gp) {
            case 1: HS2_SC(1, M3, 256);
            case 2: HS2_SC(2, M3, 256);
            case 4: HS2_SC(4, M3, 256);
            case 8: HS2_SC(8, M3, 256);
            case 16: HS2_SC(16, M3, 256);
            case 32: HS2_SC(32, M3, 256);
            case 64: HS2_SC(64, M3, 256);
            case 128: HS2_SC(128, M3, 256);
        }
    }
#undef HS2_SC
    return cudaErrorNotSupported;
}

bool scores_tc5_supported(const Params &p, hs2_dtype dt)
{
    if (padded_group(p.G, p.D) == 0) return false;
    return p.D == 256 ? full_attn_tc5_supported(p, dt) : full_tc5_supported(p, dt);
}

// shape test only (no driver query): workspace sizes must not depend on the machine
bool scores_filter_supported(const Params &p, hs2_dtype dt)
{
    auto m8 = [](int64_t x) { return x % 8 == 0 && x > 0; };
    return (p.G == 4 || p.G == 8 || p.G == 16) && dt == HS2_BF16 && p.D == HD && m8(p.qs_b) && m8(p.qs_t) && m8(p.qs_h) &&
           m8(p.ks_b) && m8(p.ks_t) && m8(p.ks_h) && (int64_t)p.B * p.Hq <= 65535;
}

// Returns cudaErrorNotSupported when the launch cannot be set up (the caller then takes the mma.sync sweep).
cudaError_t launch_scores_tc5(const Params &p, const void *Q, const void *K, const float *LSE, float *out,
                              int64_t out_stride, int64_t row0, int64_t n_rows, bool all_visible, cudaStream_t st)
{
    if (n_rows == 0) return cudaSuccess;
    if (all_visible) {   // keys a query cannot see read -inf
        const int64_t n = n_rows * out_stride;
        const int64_t fb = (n + 255) / 256;
        k_fill_tc5<<<(unsigned)(fb < 148 * 16 ? fb : 148 * 16), 256, 0, st>>>(out, n, -INFINITY);
        count_launch();
    }
    return launch_sc_mode<SC_STRIP>(p, Q, K, LSE, out, out_stride, row0, n_rows, all_visible, 1, FilterBuf{}, st);
}

// Scores of every `samp`-th key tile, written compactly: sampled tile t at columns 128 t .. 128 t + 127.
cudaError_t launch_scores_sampled_tc5(const Params &p, const void *Q, const void *K, const float *LSE, float *out,
                                      int64_t out_stride, int64_t row0, int64_t n_rows, int samp, cudaStream_t st)
{
    return launch_sc_mode<SC_SAMPLE>(p, Q, K, LSE, out, out_stride, row0, n_rows, false, samp, FilterBuf{}, st);
}

// Ordered candidate lists: every (score, key) whose order key is >= tau_key[row], in key order.
cudaError_t launch_scores_filter_tc5(const Params &p, const void *Q, const void *K, const float *LSE, int64_t row0,
                                     int64_t n_rows, const uint32_t *tau_key, void *cand, int *count,
                                     int cap, cudaStream_t st)
{
    FilterBuf fb{tau_key, static_cast<int2 *>(cand), count, cap};
    return launch_sc_mode<SC_FILTER>(p, Q, K, LSE, nullptr, 0, row0, n_rows, false, 1, fb, st);
}

// Device error word of the tcgen05 kernels (0 = no bounded wait ever ran out).  Synchronises the device.
cudaError_t read_tc5_error(unsigned *out)
{
    return cudaMemcpyFromSymbol(out, g_tc5_error, sizeof(unsigned));
}

}  // namespace hs2
