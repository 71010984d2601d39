// Sparse attention over idx ∪ window for large head groups on the 5th-generation tensor cores
// (Section 3.3: the sparse layers attend to the selected tokens plus the sliding window; Table 1: the
// paper's own models share one KV head among 64 query heads of dimension 256).
//
// With G = 64 heads per KV head every gathered key row is used by 64 heads, i.e. 64 flop per byte: the
// gather tile is a dense contraction and belongs on tcgen05.  One CTA = one (sequence, KV head, query):
//   rows of the MMA (M = 128, TMEM lane) = the G heads of the group (lanes >= G hold don't-care rows),
//   columns = 64 gathered keys per tile.
//   warps 5-7  gather producers: slot s of the virtual array [idx row | window] -> key index -> the key's
//              K and V rows copied with 16-byte cp.async into the 128-byte-swizzled UMMA operand layout
//              (void slots are zero filled), 2-stage ring, then a generic->async proxy fence and an
//              mbarrier arrive per thread.  Q (G rows) arrives by TMA.
//   warp 4     MMA issuer: S = Q K^T (M128 N64 K=D) into one of two TMEM buffers, O += P V (V MN-major).
//   warps 0-3  one thread per head: online softmax in the base-2 domain exactly as in the full-attention
//              kernel, void slots masked by a 64-bit validity word, optional sink logit in the denominator.
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
constexpr int kThreads = 256;
constexpr int kFirstProducerWarp = 5;
constexpr int kProducers = 96;
constexpr uint32_t kBarBytes = 128;
constexpr uint32_t kAlignSlack = 896;
constexpr float kRescaleThreshold = 8.f;   // log2 units

template <int D>
struct SpCfg {
    static constexpr int NQ = D / 64;                           // 64-dim slices of an operand tile
    static constexpr int CH = D / 8;                            // 16-byte chunks per row
    static constexpr uint32_t kQBytes = NQ * BM * 128;
    static constexpr uint32_t kKVStage = NQ * BN * 128;
    static constexpr uint32_t kOffQ = 0;
    static constexpr uint32_t kOffK = kOffQ + kQBytes;
    static constexpr uint32_t kOffV = kOffK + 2 * kKVStage;
    static constexpr uint32_t kOffP = kOffV + 2 * kKVStage;     // 128 rows x 64 keys bf16
    static constexpr uint32_t kOffKey = kOffP + BM * 128;       // int[2][64]: key index per slot of a stage
    static constexpr uint32_t kOffMask = kOffKey + 512;         // uint32[2][2]: validity bits of a stage
    static constexpr uint32_t kOffBar = kOffMask + 64;
    static constexpr uint32_t kSmemBytes = kOffBar + kBarBytes + kAlignSlack;
    static constexpr uint32_t kTmem = D <= 128 ? 256 : 512;     // 2 x 64 score columns + D output columns
    static constexpr int kMinBlocks = D <= 128 ? 2 : 1;
};

enum Bar { Q_FULL = 0, KV_FULL0, KV_FULL1, KV_EMPTY0, KV_EMPTY1, S_FULL0, S_FULL1, S_FREE0, S_FREE1, P_FULL, PV_DONE, N_BARS };

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    return tc5::mbar_wait(bar, parity, abort_flag, &g_sptc5_error);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
// barrier over the producer threads that also ANDs a predicate (named barrier 1)
__device__ __forceinline__ bool producers_all(bool pred)
{
    uint32_t out;
    asm volatile("{\n .reg .pred p, q;\n setp.ne.b32 p, %1, 0;\n barrier.cta.red.and.pred q, 1, %2, p;\n selp.u32 %0, 1, 0, q;\n}\n"
                 : "=r"(out) : "r"((uint32_t)pred), "n"(kProducers) : "memory");
    return out != 0;
}

template <int D>
__global__ void __launch_bounds__(kThreads, SpCfg<D>::kMinBlocks)
k_sparse_tc5(const __grid_constant__ CUtensorMap tmQ, const Params p, const __nv_bfloat16 *__restrict__ K,
             const __nv_bfloat16 *__restrict__ V, const int32_t *__restrict__ idx, const float *__restrict__ sink,
             __nv_bfloat16 *__restrict__ O, float *__restrict__ LSE)
{
    using C = SpCfg<D>;
    constexpr int NQ = C::NQ, CH = C::CH;
    constexpr uint32_t kKVStage = C::kKVStage;
    extern __shared__ char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    if (pad > kAlignSlack) {
        if (threadIdx.x == 0) atomicOr(&g_sptc5_error, 2u);
        return;
    }
    char *smem = smem_raw + pad;
    const uint32_t sbase = raw + pad;
    const uint32_t bars = sbase + C::kOffBar;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::kOffBar + N_BARS * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::kOffBar + N_BARS * 8 + 4);
    int *s_key = reinterpret_cast<int *>(smem + C::kOffKey);
    uint32_t *s_mask = reinterpret_cast<uint32_t *>(smem + C::kOffMask);
    auto bar = [&](int i) { return bars + 8u * i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t item = blockIdx.x;                 // (b, g, i) flattened
    const int i = (int)(item % p.Lq);
    const int bg = (int)(item / p.Lq);
    const int gkv = bg % p.Hkv, b = bg / p.Hkv;
    const int kvl = kvlen_of(p, b);
    const int pos = pos_of(p, b, i);
    const int nblk = (p.k + p.w + BN - 1) / BN;      // tiles of the virtual slot array [idx row | window]
    const int n_soft_warps = (p.G + 31) / 32;

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar(Q_FULL), 1);
        mbar_init(bar(KV_FULL0), kProducers); mbar_init(bar(KV_FULL1), kProducers);
        mbar_init(bar(KV_EMPTY0), 1); mbar_init(bar(KV_EMPTY1), 1);
        mbar_init(bar(S_FULL0), 1); mbar_init(bar(S_FULL1), 1);
        mbar_init(bar(S_FREE0), 32 * n_soft_warps); mbar_init(bar(S_FREE1), 32 * n_soft_warps);
        mbar_init(bar(P_FULL), 32 * n_soft_warps);
        mbar_init(bar(PV_DONE), 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(C::kTmem) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp >= kFirstProducerWarp) {
        // ------------------------------------------------ gather producers
        const int ptid = tid - kFirstProducerWarp * 32;
        const char *Kb = reinterpret_cast<const char *>(K + b * p.ks_b + gkv * p.ks_h);
        const char *Vb = reinterpret_cast<const char *>(V + b * p.ks_b + gkv * p.ks_h);
        const int64_t row_bytes = p.ks_t * 2;
        const int32_t *irow = (p.k > 0 && idx) ? idx + (((int64_t)b * p.Hkv + gkv) * p.Lq + i) * p.k : nullptr;
        if (ptid == 0 && nblk > 0) {
            mbar_expect_tx(bar(Q_FULL), (uint32_t)(NQ * p.G * 128));
#pragma unroll
            for (int sl = 0; sl < NQ; ++sl) tma_load_4d(sbase + C::kOffQ + sl * BM * 128, &tmQ, bar(Q_FULL), 64 * sl, gkv * p.G, i, b);
        }
        int issued = 0, arrived = 0;   // tiles copied / tiles handed over
        for (int t = 0; t < nblk; ++t) {
            const int st = t & 1;
            if (t > 0) {
                // hand the previous tile to the tensor core BEFORE waiting for this stage to drain: the stage is
                // released by P V of tile t-2, which the issuer orders after Q K^T of tile t-1
                cp_async_wait<0>();
                fence_proxy_async();
                mbar_arrive(bar(KV_FULL0 + ((t - 1) & 1)));
                arrived = t;
            }
            const bool ok = __all_sync(0xffffffffu, mbar_wait(bar(KV_EMPTY0 + st), ((t >> 1) & 1) ^ 1, abort_flag));
            if (ok && ptid < BN) {   // warps 5 and 6: one slot each
                const int s = t * BN + ptid;
                int j = -1;
                if (s < p.k) {
                    j = irow ? __ldg(irow + s) : -1;
                    if (j > pos - p.w || j >= kvl) j = -1;
                } else if (s < p.k + p.w) {
                    j = pos - p.w + 1 + (s - p.k);
                    if (j > pos || j >= kvl) j = -1;
                }
                s_key[st * BN + ptid] = j;
                const uint32_t m = __ballot_sync(0xffffffffu, j >= 0);
                if (lane == 0) s_mask[st * 2 + (ptid >> 5)] = m;
            }
            if (!producers_all(ok)) break;   // also publishes the key indices to the other producer threads
            const uint32_t kdst = sbase + C::kOffK + st * kKVStage, vdst = sbase + C::kOffV + st * kKVStage;
            for (int e = ptid; e < 2 * BN * CH; e += kProducers) {
                const int isv = e / (BN * CH);
                const int r = (e / CH) % BN, c = e % CH;
                const int j = s_key[st * BN + r];
                const char *src = (isv ? Vb : Kb) + (j >= 0 ? (int64_t)j * row_bytes + c * 16 : 0);
                const uint32_t dst = (isv ? vdst : kdst) + (c >> 3) * (BN * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4);
                cp_async16(dst, src, j >= 0 ? 16 : 0);
            }
            cp_async_commit();
            issued = t + 1;
        }
        cp_async_wait<0>();   // also on the abort path: nothing stays in flight
        if (issued > arrived) {
            fence_proxy_async();
            mbar_arrive(bar(KV_FULL0 + ((issued - 1) & 1)));
        }
        if (ptid == 0 && nblk > 0 && *abort_flag)
            for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar(Q_FULL), 0); ++it) {}
    } else if (warp == 4) {
        // ------------------------------------------------ MMA issuer
        if (elect_one() && nblk > 0) {
            constexpr uint32_t idS = idesc(BM, BN, 0), idPV = idesc(BM, D, 1);
            bool ok = mbar_wait(bar(Q_FULL), 0, abort_flag);
            auto issue_s = [&](int j) -> bool {
                const int st = j & 1, ph = (j >> 1) & 1;
                if (!mbar_wait(bar(KV_FULL0 + st), ph, abort_flag)) return false;
                if (!mbar_wait(bar(S_FREE0 + st), ph ^ 1, abort_flag)) return false;
                tc_fence_after();
                const uint32_t qa = sbase + C::kOffQ, ka = sbase + C::kOffK + st * kKVStage;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks & 3) * 32;
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
                if (!mbar_wait(bar(P_FULL), j & 1, abort_flag)) break;
                tc_fence_after();
                const int st = j & 1;
                const uint32_t pa = sbase + C::kOffP, va = sbase + C::kOffV + st * kKVStage;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t da = smem_desc(pa + kk * 32, 16, 1024);
                    const uint64_t db = smem_desc(va + kk * 2048, BN * 128, 1024);
                    umma(tmem + 2 * BN, da, db, idPV, (j > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bar(KV_EMPTY0 + st));
                umma_commit(bar(PV_DONE));
            }
        }
    } else if (warp < n_soft_warps) {
        // ------------------------------------------------ softmax: one thread per head of the group
        const int row = tid;
        const bool real = row < p.G;
        const int h = gkv * p.G + (real ? row : 0);
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        float m_used = -INFINITY, l = 0.f;
        if (sink && real) {   // Section 3.3 variant with a learnable sink logit: it only joins the denominator
            m_used = sink[h] * kLog2e;
            l = 1.f;
        }
        bool alive = true;
        for (int j = 0; j < nblk && alive; ++j) {
            const int sb = j & 1;
            if (!__all_sync(0xffffffffu, mbar_wait(bar(S_FULL0 + sb), (j >> 1) & 1, abort_flag))) { alive = false; break; }
            // direct acquire of the producers' validity bits (the phase is complete already)
            if (!__all_sync(0xffffffffu, mbar_wait(bar(KV_FULL0 + sb), (j >> 1) & 1, abort_flag))) { alive = false; break; }
            tc_fence_after();
            const uint32_t v0 = s_mask[sb * 2], v1 = s_mask[sb * 2 + 1];
            float s[64];
            tmem_ld32(lane_base + sb * BN, *reinterpret_cast<float (*)[32]>(&s[0]));
            tmem_ld32(lane_base + sb * BN + 32, *reinterpret_cast<float (*)[32]>(&s[32]));
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar(S_FREE0 + sb));
            float m_raw = -INFINITY;
            if ((v0 & v1) != 0xffffffffu) {
#pragma unroll
                for (int e = 0; e < 64; ++e) {
                    if (!(((e < 32 ? v0 : v1) >> (e & 31)) & 1u)) s[e] = -INFINITY;
                    m_raw = fmaxf(m_raw, s[e]);
                }
            } else {
#pragma unroll
                for (int e = 0; e < 64; ++e) m_raw = fmaxf(m_raw, s[e]);
            }
            const float m_blk = m_raw * p.scale_log2;
            const bool need = m_blk > m_used + kRescaleThreshold;
            const float m_new = need ? m_blk : m_used;
            const float corr = need ? exp2f(m_used - m_new) : 1.f;
            if (j > 0) {
                if (!__all_sync(0xffffffffu, mbar_wait(bar(PV_DONE), (j - 1) & 1, abort_flag))) { alive = false; break; }
                tc_fence_after();
                if (__any_sync(0xffffffffu, need)) {
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        float o[32];
                        tmem_ld32(lane_base + 2 * BN + c * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] *= corr;
                        tmem_st32(lane_base + 2 * BN + c * 32, o);
                    }
                    tmem_wait_st();
                }
            }
            l *= corr;
            m_used = m_new;
            const float neg_m = m_used == -INFINITY ? 0.f : -m_used;
            uint32_t pk[32];
            float l0 = 0.f, l1 = 0.f;
#pragma unroll
            for (int e = 0; e < 64; e += 2) {
                const float p0 = exp2f(fmaf(s[e], p.scale_log2, neg_m));
                const float p1 = exp2f(fmaf(s[e + 1], p.scale_log2, neg_m));
                l0 += p0; l1 += p1;
                pk[e >> 1] = pack_bf16(p0, p1);
            }
            l += l0 + l1;
            char *prow_ptr = smem + C::kOffP + row * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4 *>(prow_ptr + ((c ^ (row & 7)) << 4)) = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(P_FULL));
        }
        // ------------------------------------------------ epilogue
        bool have_o = alive && nblk > 0;
        if (have_o) have_o = mbar_wait(bar(PV_DONE), (nblk - 1) & 1, abort_flag);
        have_o = __all_sync(0xffffffffu, have_o);
        tc_fence_after();
        const bool any = l > 0.f && m_used != -INFINITY;
        const float inv = any ? 1.f / l : 0.f;
        __nv_bfloat16 *orow = O + b * p.os_b + (int64_t)i * p.os_t + h * p.os_h;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            float o[32];
            if (have_o) {
                tmem_ld32(lane_base + 2 * BN + c * 32, o);
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) o[e] = 0.f;
            }
            if (real) {
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
        if (real && LSE) LSE[((int64_t)b * p.Hq + h) * p.Lq + i] = (have_o && any) ? (m_used + log2f(l)) * kLn2 : -INFINITY;
    }
    // ------------------------------------------------ teardown
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(C::kTmem) : "memory");
    }
}

template <int D>
cudaError_t launch_sp(const Params &p, const void *Q, const void *K, const void *V, const int32_t *idx, const float *sink,
                      void *O, float *LSE, cudaStream_t st)
{
    CUtensorMap tmQ;
    if (!make_tile_map(&tmQ, Q, p.B, p.Lq, p.Hq, p.qs_b, p.qs_t, p.qs_h, 1, p.G, D)) return cudaErrorNotSupported;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!(dev >= 0 && dev < 64 && attr_set[dev])) {
        if ((e = cudaFuncSetAttribute(k_sparse_tc5<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SpCfg<D>::kSmemBytes)) != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    const int64_t items = (int64_t)p.B * p.Hkv * p.Lq;
    if (items <= 0) return cudaSuccess;
    k_sparse_tc5<D><<<(unsigned)items, kThreads, SpCfg<D>::kSmemBytes, st>>>(
        tmQ, p, (const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, idx, sink, (__nv_bfloat16 *)O, LSE);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

// bf16, head_dim 128 or 256, more than 8 and at most 128 query heads per KV head
bool sparse_tc5_supported(const Params &p, hs2_dtype dt)
{
    auto m8 = [](int64_t x) { return x % 8 == 0 && x > 0; };
    if (p.ks_t * 2 > 0x7fffffffLL) return false;
    return dt == HS2_BF16 && (p.D == 128 || p.D == 256) && p.G > 8 && p.G <= 128 && m8(p.qs_b) && m8(p.qs_t) && m8(p.qs_h) &&
           m8(p.ks_b) && m8(p.ks_t) && m8(p.ks_h) && m8(p.os_b) && m8(p.os_t) && m8(p.os_h) &&
           (int64_t)p.B * p.Hkv * p.Lq <= 0x7fffffffLL && p.k + p.w > 0 && tma_available();
}

// Returns cudaErrorNotSupported when the tensor map cannot be built (the caller then takes the generic kernel).
cudaError_t launch_sparse_tc5(const Params &p, const void *Q, const void *K, const void *V, const int32_t *idx,
                              const float *sink, void *O, float *LSE, cudaStream_t st)
{
    if (p.D == 128) return launch_sp<128>(p, Q, K, V, idx, sink, O, LSE, st);
    if (p.D == 256) return launch_sp<256>(p, Q, K, V, idx, sink, O, LSE, st);
    return cudaErrorNotSupported;
}

cudaError_t read_sparse_tc5_error(unsigned *out)
{
    return cudaMemcpyFromSymbol(out, g_sptc5_error, sizeof(unsigned));
}

}  // namespace hs2
