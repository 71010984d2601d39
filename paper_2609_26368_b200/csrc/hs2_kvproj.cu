// Producer of the KV caches the attention kernels read: C = H W^T on the 5th-generation tensor cores
// (Section 3.2, KV Bridging: K_j = Proj^K_j(H_i), V_j = Proj^V_j(H_i); one hidden-state source may feed the
// projections of several full-attention layers, which is simply more output columns).
//
//   H [T, d_model] bf16 (tokens x hidden), W [N, d_model] bf16 (one row per output feature, the layout of a linear
//   layer's weight), C [T, N]: token-major rows with a caller-given row stride, i.e. written straight into a cache
//   [.., tokens, n_kv_heads, head_dim] or a slice of a fused one.  Output either bf16, or - for the FP8 cache of the
//   sparse layers - e4m3 codes plus one fp32 scale per (token, group of 128 columns = one head), quantised in the
//   epilogue while the accumulator row is still in registers.
//
// Persistent CTAs (one per SM) walk the 128 x 256 output tiles, n-tiles fastest so that neighbouring CTAs share an H
// tile in L2: warp 4 feeds H and W tiles by TMA (64 k-columns per stage, 128-byte swizzle, 4-stage ring that runs on
// across tiles), warp 5 issues tcgen05.mma (M128 N256 K16) into one of two 256-column TMEM accumulators, warps 0-3
// (thread = output row) run the epilogue of tile i while the tensor core is already on tile i+1.  Every mbarrier
// wait is bounded.
#include <cuda.h>

#include "hs2_common.cuh"
#include "hs2_tc5.cuh"

namespace hs2 {

__device__ unsigned g_kvproj_error;   // bit 0: an mbarrier wait ran out; bit 1: shared-memory base not alignable

namespace {

using namespace tc5;

constexpr int BM = 128, BN = 256, BK = 64;
#ifndef HS2_KVP_PAIR
#define HS2_KVP_PAIR 1    // CTA pairs (cta_group::2) on 256 x 256 tiles; 0: one CTA per 128 x 256 tile
#endif
#ifndef HS2_KVP_STAGES
#define HS2_KVP_STAGES 4
#endif
constexpr int kStages = HS2_KVP_STAGES;
constexpr int kThreads = 192;
constexpr uint32_t kABytes = BM * BK * 2, kBBytes = BN * BK * 2, kStage = kABytes + kBBytes;
constexpr uint32_t kOffBar = kStages * kStage;
constexpr uint32_t kAlignSlack = 896;
constexpr uint32_t kSmemBytes = kOffBar + 128 + kAlignSlack;
constexpr int kQuantGroup = 128;      // columns that share a scale in the FP8 output (one head of dim 128)

enum Bar { FULL0 = 0, EMPTY0 = kStages, ACC_FULL0 = 2 * kStages, ACC_EMPTY0 = 2 * kStages + 2, N_BARS = 2 * kStages + 4 };
constexpr uint32_t kTmemCols = 2 * BN;   // two accumulators

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    return tc5::mbar_wait(bar, parity, abort_flag, &g_kvproj_error);
}
// two floats -> two e4m3 codes (round to nearest even, saturating), low byte = first argument
__device__ __forceinline__ uint32_t cvt_f32x2_e4m3(float lo, float hi)
{
    unsigned short d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;\n" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}

// Where the e4m3 output goes: the codes of token t, column group g (columns 128 g .. 128 g + 127) start at byte
// t * ldc + g * ld_group of C, their scale is scales[t * s_tok + g * s_grp].  (Packed: ld_group = 128, s_tok = N / 128,
// s_grp = 1; a cache of records holds a group's codes and its scale side by side.)
struct ScaleOut {
    float *scales;
    int64_t ld_group, s_tok, s_grp;
};

// Epilogue of one 128 x 256 accumulator for the thread that owns output row `tok`: bf16, or e4m3 codes with one scale
// per 128 columns.  `release` is called once, as soon as the last accumulator column is in registers.
template <bool FP8, class Release>
__device__ __forceinline__ void epilogue_rows(uint32_t acc, int64_t tok, int64_t T, int n0, int N, void *C, int64_t ldc,
                                      const ScaleOut so, Release release)
{
    if (!FP8) {
        __nv_bfloat16 *crow = static_cast<__nv_bfloat16 *>(C) + tok * ldc + n0;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            float v[32];
            tmem_ld32(acc + c * 32, v);
            tmem_wait_ld();
            if (c == BN / 32 - 1) {   // the accumulator may be overwritten by the tile after next
                tc_fence_before();
                release();
            }
            if (tok < T) {
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint4 o;
                    o.x = pack_bf16(v[8 * q4 + 0], v[8 * q4 + 1]);
                    o.y = pack_bf16(v[8 * q4 + 2], v[8 * q4 + 3]);
                    o.z = pack_bf16(v[8 * q4 + 4], v[8 * q4 + 5]);
                    o.w = pack_bf16(v[8 * q4 + 6], v[8 * q4 + 7]);
                    *reinterpret_cast<uint4 *>(crow + c * 32 + q4 * 8) = o;
                }
            }
        }
    } else {
#pragma unroll 1
        for (int grp = 0; grp < BN / kQuantGroup; ++grp) {
            const int gi = n0 / kQuantGroup + grp;   // column group of the output
            uint8_t *crow = static_cast<uint8_t *>(C) + tok * ldc + gi * so.ld_group;
            // pass 1: the group's largest magnitude; pass 2: re-read the accumulator and encode
            float amax = 0.f;
#pragma unroll 1
            for (int c = 0; c < kQuantGroup / 32; ++c) {
                float v[32];
                tmem_ld32(acc + grp * kQuantGroup + c * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) amax = fmaxf(amax, fabsf(v[e]));
            }
            const float scale = amax > 0.f ? amax / 448.f : 1.f;
            const float inv = 1.f / scale;
            if (tok < T) so.scales[tok * so.s_tok + gi * so.s_grp] = scale;
#pragma unroll 1
            for (int c = 0; c < kQuantGroup / 32; ++c) {
                float v[32];
                tmem_ld32(acc + grp * kQuantGroup + c * 32, v);
                tmem_wait_ld();
                if (grp == BN / kQuantGroup - 1 && c == kQuantGroup / 32 - 1) {
                    tc_fence_before();
                    release();
                }
                if (tok < T) {
#pragma unroll
                    for (int q4 = 0; q4 < 2; ++q4) {
                        uint32_t w4[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const float *x = v + 16 * q4 + 4 * u;
                            w4[u] = cvt_f32x2_e4m3(x[0] * inv, x[1] * inv) | (cvt_f32x2_e4m3(x[2] * inv, x[3] * inv) << 16);
                        }
                        *reinterpret_cast<uint4 *>(crow + c * 32 + q4 * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                    }
                }
            }
        }
    }
}

template <bool FP8>
__global__ void __launch_bounds__(kThreads, 1)
k_kv_project(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmW, int64_t T, int N, int dm,
             void *__restrict__ C, int64_t ldc, const ScaleOut so)
{
    extern __shared__ char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    if (pad > kAlignSlack) {
        if (threadIdx.x == 0) atomicOr(&g_kvproj_error, 2u);
        return;
    }
    char *smem = smem_raw + pad;
    const uint32_t sbase = raw + pad;
    const uint32_t bars = sbase + kOffBar;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kOffBar + N_BARS * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffBar + N_BARS * 8 + 4);
    auto bar = [&](int i) { return bars + 8u * i; };

    const int tid = threadIdx.x, warp = tid >> 5;
    const int nk = dm / BK;
    const int tiles_n = N / BN;
    const int64_t n_tiles = ((T + BM - 1) / BM) * tiles_n;

    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kStages; ++s) { mbar_init(bar(FULL0 + s), 1); mbar_init(bar(EMPTY0 + s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar(ACC_FULL0 + s), 1); mbar_init(bar(ACC_EMPTY0 + s), 128); }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        // ------------------------------------------------ TMA producer: the stage ring runs on across tiles
        if (elect_one()) {
            int c = 0, issued = 0;   // k-blocks so far
            bool ok = true;
            for (int64_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                const int n0 = (int)(tile % tiles_n) * BN;
                const int m0 = (int)(tile / tiles_n) * BM;
                for (int kb = 0; kb < nk; ++kb, ++c) {
                    const int st = c % kStages;
                    if (!mbar_wait(bar(EMPTY0 + st), ((c / kStages) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    issued = c + 1;
                    mbar_expect_tx(bar(FULL0 + st), kStage);
                    // tensors are described as [1, rows, 1, d_model]: coordinates (k, 0, row, 0)
                    tma_load_4d(sbase + st * kStage, &tmH, bar(FULL0 + st), kb * BK, 0, m0, 0);
                    tma_load_4d(sbase + st * kStage + kABytes, &tmW, bar(FULL0 + st), kb * BK, 0, n0, 0);
                }
            }
            if (*abort_flag)   // leaving early: let the copies in flight land before the CTA goes away
                for (int k2 = max(0, issued - kStages); k2 < issued; ++k2)
                    for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar(FULL0 + k2 % kStages), (k2 / kStages) & 1); ++it) {}
        }
    } else if (warp == 5) {
        // ------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t id = idesc(BM, BN, 0);
            bool ok = true;
            int c = 0, i = 0;
            for (int64_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++i) {
                const int ab = i & 1;
                if (!mbar_wait(bar(ACC_EMPTY0 + ab), ((i >> 1) & 1) ^ 1, abort_flag)) break;   // the epilogue has drained it
                tc_fence_after();
                for (int kb = 0; kb < nk; ++kb, ++c) {
                    const int st = c % kStages;
                    if (!mbar_wait(bar(FULL0 + st), (c / kStages) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t da = smem_desc(sbase + st * kStage, 16, 1024);
                    const uint64_t db = smem_desc(sbase + st * kStage + kABytes, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk)   // the descriptor's address field counts 16-byte units
                        umma(tmem + ab * BN, da + ((kk * 32) >> 4), db + ((kk * 32) >> 4), id, (kb > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(bar(EMPTY0 + st));
                }
                if (ok) umma_commit(bar(ACC_FULL0 + ab));
            }
        }
    } else {
        // ------------------------------------------------ epilogue: one thread per output row (= token)
        const int row = tid;
        bool ok = true;
        int i = 0;
        for (int64_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++i) {
            const int ab = i & 1;
            const int n0 = (int)(tile % tiles_n) * BN;
            const int64_t tok = (tile / tiles_n) * BM + row;
            const uint32_t acc = tmem + ((uint32_t)(warp * 32) << 16) + ab * BN;
            ok = __all_sync(0xffffffffu, mbar_wait(bar(ACC_FULL0 + ab), (i >> 1) & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            epilogue_rows<FP8>(acc, tok, T, n0, N, C, ldc, so, [&] { mbar_arrive(bar(ACC_EMPTY0 + ab)); });
        }
    }
    // ------------------------------------------------ teardown
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------- the same product on CTA pairs (cta_group::2)
// Two CTAs of a cluster (the two SMs of a TPC) compute one 256 x 256 output tile: CTA r holds rows 128 r .. of the H
// tile and rows 128 r .. of the W tile (i.e. output columns 128 r ..), the leader (rank 0) issues tcgen05.mma with
// .cta_group::2 (M = 256: 128 accumulator rows in each CTA's tensor memory; the W operand comes half from each CTA's
// shared memory).  Per MMA a CTA then reads 4 KB of H and 4 KB of W from its shared memory and TMA writes 8 KB into it,
// against 12 KB and 12 KB for a CTA on its own: the shared-memory traffic that held the single-CTA kernel at 73 % of
// the tensor pipe goes down by a third.  Hand-over between the two CTAs:
//   FULL[s]      in the leader: it expects the bytes of both CTAs' loads of the stage; the follower's TMA loads (no
//                multicast; .cta_group::2, which lets a load signal the peer's barrier) complete on it directly.  (A
//                first version relayed the follower's own FULL barrier through a remote mbarrier arrive per stage:
//                correct, but the arrives took over a microsecond each and the kernel 508 us instead of 205.)
//   EMPTY[s], ACC_FULL[a]  in both CTAs: tcgen05.commit from the leader with .multicast::cluster to both;
//   ACC_EMPTY[a] in the leader: its 128 epilogue threads, and one remote arrival from each of the follower's four epilogue warps.
// Every wait is bounded; the cluster barriers at both ends are reached by every thread on every path.
constexpr int kPStages = 6;
constexpr uint32_t kPHalf = 128 * BK * 2, kPStage = 2 * kPHalf;        // H rows, then W rows of this CTA
constexpr uint32_t kPOffBar = kPStages * kPStage;
enum PBar { P_FULL0 = 0, P_EMPTY0 = kPStages, P_ACC_FULL0 = 2 * kPStages, P_ACC_EMPTY0 = 2 * kPStages + 2, P_N_BARS = 2 * kPStages + 4 };
constexpr uint32_t kPSmemBytes = kPOffBar + P_N_BARS * 8 + 16 + kAlignSlack;
static_assert(kPSmemBytes <= 227 * 1024, "fits the shared memory of one SM");

__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void remote_arrive(uint32_t local_bar, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(local_bar), "r"(rank));
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];\n" ::"r"(r) : "memory");
}
__device__ __forceinline__ uint32_t peer_addr(uint32_t local, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
// TMA tile load whose completion is counted on a barrier that may live in the peer CTA of the pair
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap *tm, uint32_t bar_cluster, int c0, int c1, int c2, int c3)
{
    asm volatile("cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];\n"
                 ::"r"(dst), "l"(tm), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void umma2(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t id, uint32_t accumulate)
{
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                 ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(id), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma2_commit_both(uint32_t bar)
{
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n"
                 ::"r"(bar), "h"(mask) : "memory");
}

template <bool FP8>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
k_kv_project_pair(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmW, int64_t T, int N, int dm,
                  void *__restrict__ C, int64_t ldc, const ScaleOut so)
{
    extern __shared__ char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    if (pad > kAlignSlack) {   // (the same in both CTAs of a pair: the dynamic shared memory starts at the same offset)
        if (threadIdx.x == 0) atomicOr(&g_kvproj_error, 2u);
        return;
    }
    char *smem = smem_raw + pad;
    const uint32_t sbase = raw + pad;
    const uint32_t bars = sbase + kPOffBar;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kPOffBar + P_N_BARS * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kPOffBar + P_N_BARS * 8 + 4);
    auto bar = [&](int i) { return bars + 8u * i; };

    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t rank = cluster_rank();
    const int nk = dm / BK;
    const int tiles_n = N / 256;
    const int64_t n_tiles = ((T + 255) / 256) * tiles_n;
    const int64_t pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (tid == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kPStages; ++s) { mbar_init(bar(P_FULL0 + s), 1); mbar_init(bar(P_EMPTY0 + s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar(P_ACC_FULL0 + s), 1); mbar_init(bar(P_ACC_EMPTY0 + s), 128 + 4); }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 5) {   // both CTAs of the pair take part in the allocation
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // the peer's barriers are initialised before anything arrives on them
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        // ------------------------------------------------ TMA producer (each CTA loads its own halves)
        if (elect_one()) {
            int c = 0, issued = 0;
            bool ok = true;
            for (int64_t tile = pair; tile < n_tiles && ok; tile += n_pairs) {
                const int n0 = (int)(tile % tiles_n) * 256 + 128 * (int)rank;
                const int m0 = (int)(tile / tiles_n) * 256 + 128 * (int)rank;
                for (int kb = 0; kb < nk; ++kb, ++c) {
                    const int st = c % kPStages;
                    if (!mbar_wait(bar(P_EMPTY0 + st), ((c / kPStages) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    issued = c + 1;
                    if (rank == 0) mbar_expect_tx(bar(P_FULL0 + st), 2 * kPStage);   // this CTA's 32 KB and the follower's
                    const uint32_t full = peer_addr(bar(P_FULL0 + st), 0);          // the leader's barrier, from either CTA
                    tma_load_4d_pair(sbase + st * kPStage, &tmH, full, kb * BK, 0, m0, 0);
                    tma_load_4d_pair(sbase + st * kPStage + kPHalf, &tmW, full, kb * BK, 0, n0, 0);
                }
            }
            if (*abort_flag && rank == 0)   // leaving early: let the copies in flight land before the CTA goes away
                for (int k2 = max(0, issued - kPStages); k2 < issued; ++k2)
                    for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar(P_FULL0 + k2 % kPStages), (k2 / kPStages) & 1); ++it) {}
        }
    } else if (warp == 5) {
        if (elect_one()) {
            if (rank == 0) {
                // -------------------------------------------- MMA issuer of the pair
                constexpr uint32_t id = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
                bool ok = true;
                int c = 0, i = 0;
                for (int64_t tile = pair; tile < n_tiles && ok; tile += n_pairs, ++i) {
                    const int ab = i & 1;
                    if (!mbar_wait(bar(P_ACC_EMPTY0 + ab), ((i >> 1) & 1) ^ 1, abort_flag)) break;
                    tc_fence_after();
                    for (int kb = 0; kb < nk; ++kb, ++c) {
                        const int st = c % kPStages;
                        if (!mbar_wait(bar(P_FULL0 + st), (c / kPStages) & 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t da = smem_desc(sbase + st * kPStage, 16, 1024);
                        const uint64_t db = smem_desc(sbase + st * kPStage + kPHalf, 16, 1024);
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk)
                            umma2(tmem + ab * BN, da + ((kk * 32) >> 4), db + ((kk * 32) >> 4), id, (kb > 0 || kk > 0) ? 1u : 0u);
                        umma2_commit_both(bar(P_EMPTY0 + st));
                    }
                    if (ok) umma2_commit_both(bar(P_ACC_FULL0 + ab));
                }
            }
        }
    } else {
        // ------------------------------------------------ epilogue: one thread per output row of this CTA's half
        const int row = tid;
        bool ok = true;
        int i = 0;
        for (int64_t tile = pair; tile < n_tiles && ok; tile += n_pairs, ++i) {
            const int ab = i & 1;
            const int n0 = (int)(tile % tiles_n) * 256;
            const int64_t tok = (tile / tiles_n) * 256 + 128 * (int64_t)rank + row;
            const uint32_t acc = tmem + ((uint32_t)(warp * 32) << 16) + ab * BN;
            ok = __all_sync(0xffffffffu, mbar_wait(bar(P_ACC_FULL0 + ab), (i >> 1) & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            epilogue_rows<FP8>(acc, tok, T, n0, N, C, ldc, so, [&] {
                if (rank == 0) {
                    mbar_arrive(bar(P_ACC_EMPTY0 + ab));
                } else {
                    // one arrival per follower warp in the leader's barrier (no CTA-wide meeting point that a warp
                    // which has given up could leave the others waiting at)
                    __syncwarp();
                    if ((tid & 31) == 0) remote_arrive(bar(P_ACC_EMPTY0 + ab), 0);
                }
            });
        }
    }
    // ------------------------------------------------ teardown
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // no CTA frees tensor memory or leaves while its peer may still arrive on its barriers
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

template <bool FP8>
cudaError_t launch(int64_t T, int N, int dm, const void *H, int64_t ldh, const void *W, int64_t ldw, void *C, int64_t ldc,
                   const ScaleOut so, cudaStream_t st)
{
    CUtensorMap tmH, tmW;
    // [1, rows, 1, d_model] views: token stride ld, a single "head"
    if (!make_tile_map(&tmH, H, 1, (int)T, 1, T * ldh, ldh, ldh, BM, 1, dm) ||
        !make_tile_map(&tmW, W, 1, N, 1, (int64_t)N * ldw, ldw, ldw, BN, 1, dm))
        return cudaErrorNotSupported;
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorNotSupported;
    if (!done[dev]) {
        if ((e = cudaFuncSetAttribute(k_kv_project<FP8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes)) != cudaSuccess) return e;
        done[dev] = true;
    }
    static int n_sm[64] = {};
    if (n_sm[dev] == 0 && (e = cudaDeviceGetAttribute(&n_sm[dev], cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
#if HS2_KVP_PAIR
    {
        // CTA pairs on 256 x 256 tiles; W is loaded in halves of 128 rows
        CUtensorMap tmW2;
        if (make_tile_map(&tmW2, W, 1, N, 1, (int64_t)N * ldw, ldw, ldw, 128, 1, dm)) {
            static bool done2[64] = {};
            if (!done2[dev]) {
                if ((e = cudaFuncSetAttribute(k_kv_project_pair<FP8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPSmemBytes)) != cudaSuccess) return e;
                done2[dev] = true;
            }
            const int64_t n_tiles2 = ((T + 255) / 256) * (N / 256);
            const int64_t pairs = n_tiles2 < n_sm[dev] / 2 ? n_tiles2 : n_sm[dev] / 2;
            if (pairs >= 1) {
                k_kv_project_pair<FP8><<<(unsigned)(2 * pairs), kThreads, kPSmemBytes, st>>>(tmH, tmW2, T, N, dm, C, ldc, so);
                count_launch();
                return cudaGetLastError();
            }
        }
    }
#endif
    const int64_t n_tiles = ((T + BM - 1) / BM) * (N / BN);
    const unsigned grid = (unsigned)(n_tiles < n_sm[dev] ? n_tiles : n_sm[dev]);
    k_kv_project<FP8><<<grid, kThreads, kSmemBytes, st>>>(tmH, tmW, T, N, dm, C, ldc, so);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool kv_project_supported(int64_t T, int N, int dm, int64_t ldh, int64_t ldw, int64_t ldc, bool fp8)
{
    return T > 0 && T <= 0x7fffff00LL && N > 0 && N % BN == 0 && dm > 0 && dm % BK == 0 &&
           ldh >= dm && ldw >= dm && ldc >= N && ldh % 8 == 0 && ldw % 8 == 0 && ldc % (fp8 ? 16 : 8) == 0;
}

cudaError_t launch_kv_project(int64_t T, int N, int dm, const void *H, int64_t ldh, const void *W, int64_t ldw, void *C,
                              int64_t ldc, float *scales, cudaStream_t st)
{
    if (!tma_available()) return cudaErrorNotSupported;
    const ScaleOut so{scales, kQuantGroup, N / kQuantGroup, 1};
    return scales ? launch<true>(T, N, dm, H, ldh, W, ldw, C, ldc, so, st)
                  : launch<false>(T, N, dm, H, ldh, W, ldw, C, ldc, so, st);
}

cudaError_t launch_kv_project_records(int64_t T, int N, int dm, const void *H, int64_t ldh, const void *W, int64_t ldw,
                                      void *C, int64_t ldc, int64_t ld_group, float *scales, int64_t s_tok, int64_t s_grp,
                                      cudaStream_t st)
{
    if (!tma_available()) return cudaErrorNotSupported;
    return launch<true>(T, N, dm, H, ldh, W, ldw, C, ldc, ScaleOut{scales, ld_group, s_tok, s_grp}, st);
}

cudaError_t read_kvproj_error(unsigned *out) { return cudaMemcpyFromSymbol(out, g_kvproj_error, sizeof(unsigned)); }

}  // namespace hs2
