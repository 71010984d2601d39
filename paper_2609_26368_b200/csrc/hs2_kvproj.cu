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

template <bool FP8>
__global__ void __launch_bounds__(kThreads, 1)
k_kv_project(const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmW, int64_t T, int N, int dm,
             void *__restrict__ C, int64_t ldc, float *__restrict__ scales)
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
            if (!FP8) {
                __nv_bfloat16 *crow = static_cast<__nv_bfloat16 *>(C) + tok * ldc + n0;
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    float v[32];
                    tmem_ld32(acc + c * 32, v);
                    tmem_wait_ld();
                    if (c == BN / 32 - 1) {   // the accumulator may be overwritten by the tile after next
                        tc_fence_before();
                        mbar_arrive(bar(ACC_EMPTY0 + ab));
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
                uint8_t *crow = static_cast<uint8_t *>(C) + tok * ldc + n0;
#pragma unroll 1
                for (int grp = 0; grp < BN / kQuantGroup; ++grp) {
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
                    if (tok < T) scales[tok * (N / kQuantGroup) + (n0 + grp * kQuantGroup) / kQuantGroup] = scale;
#pragma unroll 1
                    for (int c = 0; c < kQuantGroup / 32; ++c) {
                        float v[32];
                        tmem_ld32(acc + grp * kQuantGroup + c * 32, v);
                        tmem_wait_ld();
                        if (grp == BN / kQuantGroup - 1 && c == kQuantGroup / 32 - 1) {
                            tc_fence_before();
                            mbar_arrive(bar(ACC_EMPTY0 + ab));
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
                                *reinterpret_cast<uint4 *>(crow + grp * kQuantGroup + c * 32 + q4 * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                            }
                        }
                    }
                }
            }
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

template <bool FP8>
cudaError_t launch(int64_t T, int N, int dm, const void *H, int64_t ldh, const void *W, int64_t ldw, void *C, int64_t ldc,
                   float *scales, cudaStream_t st)
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
    const int64_t n_tiles = ((T + BM - 1) / BM) * (N / BN);
    const unsigned grid = (unsigned)(n_tiles < n_sm[dev] ? n_tiles : n_sm[dev]);
    k_kv_project<FP8><<<grid, kThreads, kSmemBytes, st>>>(tmH, tmW, T, N, dm, C, ldc, scales);
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
    return scales ? launch<true>(T, N, dm, H, ldh, W, ldw, C, ldc, scales, st)
                  : launch<false>(T, N, dm, H, ldh, W, ldw, C, ldc, nullptr, st);
}

cudaError_t read_kvproj_error(unsigned *out) { return cudaMemcpyFromSymbol(out, g_kvproj_error, sizeof(unsigned)); }

}  // namespace hs2
