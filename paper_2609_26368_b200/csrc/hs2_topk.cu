// Token-level top-k outside the forced window on a materialised score row (Section 3.3).
//
// One CTA per (batch, KV head, query) row.  The row's candidates are keys 0 .. pos-w.  An exact
// radix select on order-preserving 32-bit keys (four 8-bit digits, most significant first) finds
// the value of the take-th largest score and how many candidates equal to it are still needed;
// one ordered compaction pass then writes the kept indices in ascending key order, taking equal
// scores from the lowest index upwards.  The result depends only on the score bits.
#include <cooperative_groups.h>

#include <algorithm>

#include "hs2_common.cuh"

namespace hs2 {
namespace {

#ifndef HS2_TOPK_NBT
#define HS2_TOPK_NBT 4
#endif
#ifndef HS2_TOPK_LINEAR
#define HS2_TOPK_LINEAR 1
#endif
constexpr int kItems = 4;                    // consecutive scores per thread per step
constexpr unsigned kListCap = 2048;          // threshold-bin candidates kept in shared memory (cached variant)
constexpr int kStageOut = 4096;              // selected indices of a row staged in shared memory (cached variant)

// float -> uint32 whose unsigned order is the float order; -0 is folded onto +0 first.
__device__ __forceinline__ uint32_t order_key(float f)
{
    uint32_t u = __float_as_uint(f);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <bool VEC>
__device__ __forceinline__ void load_keys(const float *row, int j0, int nc, uint32_t (&key)[kItems], bool (&ok)[kItems])
{
    if (VEC && j0 + kItems <= nc) {
        const float4 v = *reinterpret_cast<const float4 *>(row + j0);
        key[0] = order_key(v.x); key[1] = order_key(v.y); key[2] = order_key(v.z); key[3] = order_key(v.w);
        ok[0] = ok[1] = ok[2] = ok[3] = true;
    } else {
#pragma unroll
        for (int e = 0; e < kItems; ++e) {
            ok[e] = j0 + e < nc;
            key[e] = ok[e] ? order_key(row[j0 + e]) : 0u;
        }
    }
}

// Shared by both variants: find, from the top, the digit at which the running count reaches `need`.
// hist[256] is complete; warp 0 scans it.  Writes the new prefix and the remaining need.
__device__ __forceinline__ void pick_digit(const unsigned *hist, unsigned prefix, unsigned need, int lane, unsigned *s_prefix,
                                           unsigned *s_need)
{
    // lane l owns digits 255-8l .. 248-8l (descending)
    unsigned mine = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) mine += hist[255 - 8 * lane - e];
    unsigned incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    const unsigned before = incl - mine;
    if (before < need && need <= incl) {
        unsigned cum = before;
        for (int e = 0; e < 8; ++e) {
            const unsigned c = hist[255 - 8 * lane - e];
            if (cum + c >= need) {
                *s_prefix = (prefix << 8) | (unsigned)(255 - 8 * lane - e);
                *s_need = need - cum;
                break;
            }
            cum += c;
        }
    }
}

#ifndef HS2_TOPK_RANKMAX
#define HS2_TOPK_RANKMAX 64
#endif
constexpr unsigned kRankMax = HS2_TOPK_RANKMAX;           // a threshold bin this small is finished by ranking its members

// ---- rows that fit in registers: THREADS x E candidates, read once ------------------------------
// Thread t owns the E consecutive candidates E t .. E t + E - 1, so the ascending-index order of the
// output is (thread, element) order and the ordered compaction needs a single block scan.  The radix
// digits are taken below the common leading bits of the row's smallest and largest key, which makes
// the first round spread the candidates over all 256 bins (log-probabilities share their top bits).

// value of the `need`-th largest of list[0..n) (n >= need >= 1): four 8-bit rounds, CTA-wide, on a shared list
template <int THREADS>
__device__ __forceinline__ uint32_t select_on_list(const uint32_t *list, unsigned n, unsigned need, unsigned *hist,
                                                   unsigned *s_prefix, unsigned *s_need, int tid, int lane, int warp)
{
    unsigned prefix = 0;
    for (int round = 0; round < 4; ++round) {
        const int shift = 24 - 8 * round;
        if (tid < 256) hist[tid] = 0;
        if (THREADS < 256) for (int t = tid + THREADS; t < 256; t += THREADS) hist[t] = 0;
        __syncthreads();
        for (unsigned t = tid; t < n; t += THREADS) {
            const uint32_t kk = list[t];
            if (round == 0 || (kk >> (shift + 8)) == prefix) atomicAdd(&hist[(kk >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (warp == 0) pick_digit(hist, prefix, need, lane, s_prefix, s_need);
        __syncthreads();
        prefix = *s_prefix;
        need = *s_need;
        __syncthreads();
    }
    return prefix;
}

// exclusive prefix of `v` over the CTA in thread order; *total receives the sum (s_warp: WARPS words)
template <int WARPS>
__device__ __forceinline__ unsigned block_excl_scan(unsigned v, unsigned *s_warp, int lane, int warp, unsigned *total)
{
    unsigned incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();   // s_warp may still be read from an earlier use
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    unsigned wsum = lane < WARPS ? s_warp[lane] : 0u;
    unsigned wincl = wsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, wincl, o);
        if (lane >= o) wincl += t;
    }
    *total = __shfl_sync(0xffffffffu, wincl, WARPS - 1);
    return __shfl_sync(0xffffffffu, wincl - wsum, warp) + incl - v;
}

// sampled scores of a row with n candidates: every samp-th tile of 128 keys, the last one possibly partial
__host__ __device__ __forceinline__ int sample_size(int n, int samp)
{
    const int q = n / (samp * 128), rem = n - q * samp * 128;
    return q * 128 + (rem < 128 ? rem : 128);
}
// Rank (from the top) of the sample whose value is a safe lower bound of the row's take-th largest score.
// The sample holds n_s of the row's n keys; of the row's top `take` about take * n_s / n fall into it, and
// the rank is put five standard deviations above that mean (short rows sample more than 1/samp of their keys).
__device__ __forceinline__ int sample_rank(int take, int n, int n_s)
{
    const float m = (float)take * (float)n_s / (float)n;
    return (int)(m + 5.f * sqrtf(m) + 2.f);
}

__device__ __forceinline__ void topk_cp_async16(void *dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void topk_cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\n cp.async.wait_group 0;\n" ::: "memory");
}

#ifndef HS2_TOPK_STAGE
#define HS2_TOPK_STAGE 1      // rows reach the registers through a coalesced copy into shared memory
#endif
// dynamic shared memory of the two selects of the filtered path: [bitmap (candidate select only)][staged row]
__host__ __device__ inline size_t cached_bitmap_bytes(int Lk) { return ((size_t)((Lk + 31) / 32) * 4 + 15) & ~(size_t)15; }
constexpr size_t cached_stage_bytes(int threads, int e) { return (size_t)threads * (e + 4) * 4; }

template <int THREADS, int E, bool VEC>
__global__ void __launch_bounds__(THREADS, THREADS > 256 ? 1 : (E > 32 ? 2 : 3))
k_topk_cached(const Params p, const float *__restrict__ scores, int64_t score_stride, int32_t *__restrict__ idx,
              int64_t row0, int nc_lo, int nc_hi)
{
    constexpr int WARPS = THREADS / 32;
    __shared__ unsigned hist[256];
    __shared__ unsigned s_warp[WARPS];
    __shared__ unsigned s_min[WARPS];   // per-warp partial of the row-wide reduction
    __shared__ unsigned s_prefix, s_need, s_cnt;
    __shared__ uint32_t s_list[kListCap];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row = row0 + blockIdx.x;   // (b, g, i), i fastest
    const int i = (int)(row % p.Lq);
    const int b = (int)(row / ((int64_t)p.Lq * p.Hkv));
    const int kvl = kvlen_of(p, b);
    const int pos = pos_of(p, b, i);
    const int n_keys = max(0, min(pos - p.w + 1, kvl));   // the row's candidates are keys 0..n_keys-1
    const int k_row = min(p.k, n_keys);                   // how many of them are selected
    const int nc = n_keys, take = k_row;
    if (nc <= nc_lo || nc > nc_hi) return;   // this row belongs to another variant's launch
    int32_t *out = idx + row * p.k;
    const float *srow = scores + (int64_t)blockIdx.x * score_stride;

    if (k_row == n_keys) {   // every candidate is kept: no need to look at the scores
        for (int t = tid; t < p.k; t += THREADS) out[t] = t < n_keys ? t : -1;
        return;
    }
    const int j0 = tid * E;
    const int nv = min(max(nc - j0, 0), E);   // this thread's slots 0 .. nv-1 hold candidates
    const bool has = nv > 0;   // threads (whole warps, on short rows) past the row's end skip every per-candidate loop
    uint32_t key[E];
    // which bits differ anywhere in the row: OR of (key ^ key of candidate 0), one logic op per candidate
    const uint32_t ref = order_key(__ldg(srow));
    unsigned diff = 0u;
    if (has)
#pragma unroll
    for (int e4 = 0; e4 < E; e4 += 4) {
        if (VEC && j0 + e4 + 4 <= nc) {
            const float4 v = __ldg(reinterpret_cast<const float4 *>(srow + j0 + e4));
            key[e4] = order_key(v.x); key[e4 + 1] = order_key(v.y); key[e4 + 2] = order_key(v.z); key[e4 + 3] = order_key(v.w);
#pragma unroll
            for (int e = e4; e < e4 + 4; ++e) diff |= key[e] ^ ref;
        } else {
#pragma unroll
            for (int e = e4; e < e4 + 4; ++e) {
                const bool ok = e < nv;
                key[e] = ok ? order_key(srow[j0 + e]) : 0u;
                if (ok) diff |= key[e] ^ ref;
            }
        }
    }
    else {
#pragma unroll
        for (int e = 0; e < E; ++e) key[e] = 0u;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) diff |= __shfl_xor_sync(0xffffffffu, diff, o);
    if (lane == 0) s_min[warp] = diff;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < WARPS; ++w) diff |= s_min[w];

    // bits above `hi` are equal in every candidate; resolve the rest 8 bits at a time
    int hi = 32 - __clz(diff);                 // 0 when all candidates are equal
    unsigned prefix = hi >= 32 ? 0u : (ref >> hi);
    unsigned need = (unsigned)take;
    bool on_list = false;                      // later rounds run on the threshold bin's candidates only
    unsigned n_list = 0;
    bool first = true;
    while (hi > 0) {
        const int w = min(8, hi), shift = hi - w;
        const unsigned dmask = (1u << w) - 1u;
        if (tid < 256) hist[tid] = 0;
        if (THREADS < 256) for (int t = tid + THREADS; t < 256; t += THREADS) hist[t] = 0;
        __syncthreads();
        if (on_list) {
            for (unsigned t = tid; t < n_list; t += THREADS) {
                const uint32_t kk = s_list[t];
                if ((kk >> hi) == prefix) atomicAdd(&hist[(kk >> shift) & dmask], 1u);
            }
        } else if (has) {
#pragma unroll
            for (int e = 0; e < E; ++e) {
                // slots past the row's end hold key 0, which is below every real key (the lowest, -inf, maps to
                // 0x007fffff): counted or not, they sit at the very bottom of the lowest bin and are never reached
                // (in the first round every candidate has the common prefix by construction)
                const bool live = first || (key[e] >> hi) == prefix;
                if (live) atomicAdd(&hist[(key[e] >> shift) & dmask], 1u);
            }
        }
        __syncthreads();
        if (warp == 0) pick_digit(hist, prefix, need, lane, &s_prefix, &s_need);
        if (tid == 0) s_cnt = 0;
        __syncthreads();
        // pick_digit composes (prefix << 8) | digit; rebuild with the real digit width
        const unsigned digit = s_prefix & 255u;
        const unsigned in_bin = hist[digit];
        prefix = (hi >= 32 ? 0u : (prefix << w)) | digit;
        need = s_need;
        hi = shift;
        first = false;
        const bool collect = !on_list && hi > 0 && in_bin <= kListCap;
        __syncthreads();   // every thread has read hist[digit] before the next round zeroes the histogram
        if (collect) {
            // every candidate that can still be the take-th largest sits in this bin (at most kListCap of them)
            // (one atomic per member on a single word looks wasteful, but a ballot-aggregated version was measured
            // slower: 2.31 vs 2.18 ms for the whole full layer on the 8K benchmark)
            if (has)
#pragma unroll
            for (int e = 0; e < E; ++e)
                if ((key[e] >> hi) == prefix) {
                    const unsigned slot = atomicAdd(&s_cnt, 1u);
                    if (slot < kListCap) s_list[slot] = key[e];
                }
            __syncthreads();
            on_list = true;
            n_list = min(s_cnt, kListCap);
            if (n_list <= kRankMax && n_list <= (unsigned)THREADS) {   // one thread per member
                // A short list is finished by ranking instead of more histogram rounds (four barriers each): member
                // t is the answer when fewer than `need` members are above it and at least `need` are not below it.
                if ((unsigned)tid < n_list) {
                    const uint32_t kt = s_list[tid];
                    unsigned gt = 0, eq = 0;
                    for (unsigned u = 0; u < n_list; ++u) {
                        const uint32_t v = s_list[u];
                        gt += v > kt;
                        eq += v == kt;
                    }
                    if (gt < need && need <= gt + eq) { s_prefix = kt; s_need = need - gt; }   // equal members write the same
                }
                __syncthreads();
                prefix = s_prefix;   // the full key
                need = s_need;
                hi = 0;
            }
        }
    }
    const uint32_t tau = diff == 0u ? ref : prefix;                  // key of the take-th largest candidate
    const unsigned need_eq = need;                                   // equal keys kept, lowest indices first

    // ---- ordered compaction with one block scan
    // which of this thread's candidates are above tau / equal to it (key 0, past the end, is below tau)
    static_assert(E <= 64, "one 64-bit mask per thread");
    unsigned long long m_gt = 0ull, m_eq = 0ull;
    if (has)
#pragma unroll
    for (int e = 0; e < E; ++e) {
        m_gt |= (unsigned long long)(key[e] > tau) << e;
        m_eq |= (unsigned long long)(key[e] == tau) << e;
    }
    const unsigned n_gt = __popcll(m_gt), n_eq = __popcll(m_eq);
    const unsigned packed = (n_gt << 16) | n_eq;   // both totals stay below 65536 (rows <= 32768)
    unsigned incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    unsigned wsum = lane < WARPS ? s_warp[lane] : 0u;
    unsigned wincl = wsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, wincl, o);
        if (lane >= o) wincl += t;
    }
    const unsigned excl = __shfl_sync(0xffffffffu, wincl - wsum, warp) + incl - packed;
    unsigned gt_before = excl >> 16, eq_before = excl & 0xffffu;
    // the kept indices are collected in shared memory (every thread owns a run of positions) and leave as one
    // coalesced row; rows with more than kStageOut selected tokens write straight to global memory
    extern __shared__ int s_out[];
    const bool staged = p.k <= kStageOut;
    int *dst = staged ? s_out : out;
    {
        // of the equal ones this thread keeps those that are still among the first need_eq of the row
        unsigned keep_eq = eq_before < need_eq ? min(n_eq, need_eq - eq_before) : 0u;
        unsigned long long m_keep = m_gt;
        while (keep_eq > 0) {   // rare: ties at the threshold
            const unsigned long long low = m_eq & (0ull - m_eq);
            m_keep |= low;
            m_eq ^= low;
            --keep_eq;
        }
        unsigned posn = gt_before + min(eq_before, need_eq);
        while (m_keep) {   // ascending candidate index
            const int e = __ffsll((long long)m_keep) - 1;
            m_keep &= m_keep - 1;
            dst[posn++] = j0 + e;
        }
    }
    if (staged) {
        __syncthreads();
        for (int t = tid; t < p.k; t += THREADS) out[t] = t < take ? s_out[t] : -1;
    } else {
        for (int t = take + tid; t < p.k; t += THREADS) out[t] = -1;
    }
}

// ---- whole rows, first round on a linear scale -------------------------------------------------------
// The scores of a row are logarithms of probabilities: as floats they spend their leading bits on the exponent,
// and most candidates share one or two exponents, so a radix digit of the float key leaves a threshold bin with a
// large share of the row (measured on the 8K benchmark: the rounds on that bin's members were 43 % of the select).
// Any monotone map to bins narrows the search just as exactly, so the first round here bins the VALUES on a linear
// scale between the row's smallest and largest score (4 bins per thread); the threshold bin's members - now a few
// dozen - go to a shared list as order-preserving keys and the exact take-th largest is found there (by ranking
// when the list is short, else by the radix select on the list).  The candidates stay in registers as floats;
// key equality and float equality agree (-0 and +0 are one key; NaN scores are a caller error).  Slots past the
// row's end hold -inf and, having the highest indices, lose every tie, so they can never be selected while
// take <= candidates.  A row whose range is empty or not finite puts every candidate in one bin: slow, still exact.
// v > t and v == t as 0/1, comparing denormals as they are (the file is compiled with flush-to-zero, which would
// make every denormal score equal to zero in a plain comparison; the keys, and the oracle, tell them apart)
__device__ __forceinline__ void compare_exact(float v, float t, unsigned &gt, unsigned &eq)
{
    asm("{\n .reg .pred p, q;\n setp.gt.f32 p, %2, %3;\n setp.eq.f32 q, %2, %3;\n selp.u32 %0, 1, 0, p;\n selp.u32 %1, 1, 0, q;\n}\n"
        : "=r"(gt), "=r"(eq) : "f"(v), "f"(t));
}

__device__ __forceinline__ unsigned ge_exact(float v, float t)
{
    unsigned r;
    asm("{\n .reg .pred p;\n setp.ge.f32 p, %1, %2;\n selp.u32 %0, 1, 0, p;\n}\n" : "=r"(r) : "f"(v), "f"(t));
    return r;
}

#ifndef HS2_TOPK_MINB32
#define HS2_TOPK_MINB32 4
#endif
#ifndef HS2_TOPK_ROWS
#define HS2_TOPK_ROWS 1    // rows per CTA of the linear kernel (consecutive queries of one (sequence, KV head))
#endif
#ifndef HS2_TOPK_WIDE
#define HS2_TOPK_WIDE 1    // rows of 8193..16384 candidates: 32 per thread on 512 threads, two CTAs per SM (4 % faster than 64 per
                           // thread on 256; the same step for the longest class, 1024 threads, measured 5 % slower)
#endif
// one row of k_topk_linear; every exit is taken by the whole CTA
template <int THREADS, int E, bool VEC>
__device__ __forceinline__ void topk_linear_row(const Params &p, const float *__restrict__ scores, int64_t score_stride,
                                                int32_t *__restrict__ idx, int64_t row0, int nc_lo, int nc_hi, int64_t row)
{
    constexpr int WARPS = THREADS / 32;
    constexpr int NBT = HS2_TOPK_NBT;       // bins per thread
    constexpr int NB = NBT * THREADS;       // bins of the first round
    __shared__ unsigned hist[NB < 256 ? 256 : NB];
    __shared__ unsigned s_warp[WARPS];
    __shared__ float s_lo[WARPS], s_hi[WARPS];
    __shared__ unsigned s_prefix, s_need, s_cnt, s_bin, s_eq;
    extern __shared__ int s_dyn[];          // [selected indices staged for the coalesced store][list: THREADS * E keys]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t local = row - row0;
    const int i = (int)(row % p.Lq);
    const int b = (int)(row / ((int64_t)p.Lq * p.Hkv));
    const int kvl = kvlen_of(p, b);
    const int pos = pos_of(p, b, i);
    const int nc = max(0, min(pos - p.w + 1, kvl));   // the row's candidates are keys 0..nc-1
    const int take = min(p.k, nc);                    // how many of them are selected
    if (nc <= nc_lo || nc > nc_hi) return;            // this row belongs to another variant's launch
    int32_t *out = idx + row * p.k;
    const float *srow = scores + local * score_stride;
    if (take == nc) {   // every candidate is kept: no need to look at the scores
        for (int t = tid; t < p.k; t += THREADS) out[t] = t < nc ? t : -1;
        return;
    }
    const bool staged = p.k <= kStageOut;
    int *s_out = s_dyn;
    uint32_t *s_list = reinterpret_cast<uint32_t *>(s_dyn + (staged ? p.k : 0));

    const int j0 = tid * E;
    const bool has = j0 < nc;   // threads (whole warps, on short rows) past the row's end skip every per-candidate loop
    constexpr int CPT = E / 4;  // 16-byte chunks per thread
#if HS2_TOPK_STAGE
    // A thread's candidates are E consecutive floats, so its own 16-byte loads would sit E * 4 bytes apart between
    // lanes: 32 cache lines per warp instruction.  Instead consecutive lanes copy consecutive chunks into the (still
    // unused) list, chunk c at slot c + c / CPT, and every thread then reads its chunks at a pitch of CPT + 1 slots:
    // both sides are free of bank conflicts.  (Fetching the NEXT row this way during the current one, a CTA taking
    // 16 consecutive queries, was also built: no faster than this, so the load's cost was its access pattern.)
    float *s_stage = reinterpret_cast<float *>(s_dyn + (((staged ? p.k : 0) + 3) & ~3));
    if (VEC) {
#pragma unroll
        for (int it = 0; it < CPT; ++it) {
            const int c = it * THREADS + tid;
            if (4 * c + 4 <= nc) topk_cp_async16(s_stage + (c + c / CPT) * 4, srow + 4 * c);
        }
        topk_cp_async_wait_all();
        __syncthreads();
    }
    constexpr bool from_stage = VEC;
#else
    constexpr bool from_stage = false;
    float *s_stage = nullptr;
#endif
    float val[E];
    float vmin = INFINITY, vmax = -INFINITY;
    if (has)
#pragma unroll
    for (int e4 = 0; e4 < E; e4 += 4) {
        if (VEC && j0 + e4 + 4 <= nc) {
            const float4 v = from_stage ? *reinterpret_cast<const float4 *>(s_stage + ((CPT + 1) * tid + (e4 >> 2)) * 4)
                                        : __ldg(reinterpret_cast<const float4 *>(srow + j0 + e4));
            val[e4] = v.x; val[e4 + 1] = v.y; val[e4 + 2] = v.z; val[e4 + 3] = v.w;
            vmin = fminf(fminf(vmin, v.x), fminf(v.y, fminf(v.z, v.w)));
            vmax = fmaxf(fmaxf(vmax, v.x), fmaxf(v.y, fmaxf(v.z, v.w)));
        } else {
#pragma unroll
            for (int e = e4; e < e4 + 4; ++e) {
                const bool ok = j0 + e < nc;
                val[e] = ok ? srow[j0 + e] : -INFINITY;
                if (ok) { vmin = fminf(vmin, val[e]); vmax = fmaxf(vmax, val[e]); }
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        vmin = fminf(vmin, __shfl_xor_sync(0xffffffffu, vmin, o));
        vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, o));
    }
    if (lane == 0) { s_lo[warp] = vmin; s_hi[warp] = vmax; }
#pragma unroll
    for (int t = 0; t < NBT; ++t) hist[t * THREADS + tid] = 0u;
    if (tid == 0) s_cnt = 0u;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < WARPS; ++w) { vmin = fminf(vmin, s_lo[w]); vmax = fmaxf(vmax, s_hi[w]); }
    // bin(v) = clamp(floor(v * c + d), 0, NB - 1) with one fused multiply-add: monotone in v, and the same
    // instruction in both passes gives the same bin
    const float range = vmax - vmin;
    const bool flat = !(range > 0.f) || !(range < 3.0e38f);
    const float c = flat ? 0.f : (float)NB / range;
    const float d = flat ? 0.f : -vmin * c;
    // (the conversion to unsigned saturates: negative values, -inf and NaN give bin 0)
    auto bin_of = [&](float v) { return min(__float2uint_rd(__fmaf_rn(v, c, d)), (unsigned)(NB - 1)); };
    if (has)
#pragma unroll
    for (int e = 0; e < E; ++e) atomicAdd(&hist[bin_of(val[e])], 1u);
    __syncthreads();
    // from the top: the bin at which the running count reaches `take`.  Thread t owns bins NB-1-NBT*t-e.
    unsigned mine = 0;
#pragma unroll
    for (int e = 0; e < NBT; ++e) mine += hist[NB - 1 - NBT * tid - e];
    unsigned total;
    const unsigned before = block_excl_scan<WARPS>(mine, s_warp, lane, warp, &total);
    if (before < (unsigned)take && (unsigned)take <= before + mine) {
        unsigned cum = before;
#pragma unroll
        for (int e = 0; e < NBT; ++e) {
            const unsigned cnt = hist[NB - 1 - NBT * tid - e];
            if (cum < (unsigned)take && (unsigned)take <= cum + cnt) { s_bin = NB - 1 - NBT * tid - e; s_need = (unsigned)take - cum; }
            cum += cnt;
        }
    }
    __syncthreads();
    const unsigned tbin = s_bin;
    unsigned need = s_need;
    // the threshold bin's members, as keys
    // (bin_of(v) == tbin as a range test on the same fused multiply-add: floor(x) == tbin; the clamped ends are open:
    // nothing is below -inf, and no comparison with NaN holds, so bin 0 takes NaN and -inf, the last bin +inf)
    const float x_lo = tbin == 0u ? -INFINITY : (float)tbin;
    const float x_hi = tbin == (unsigned)(NB - 1) ? __uint_as_float(0x7fc00000u) : (float)(tbin + 1u);
    if (has)
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const float x = __fmaf_rn(val[e], c, d);
        if (!(x < x_lo) && !(x >= x_hi)) s_list[atomicAdd(&s_cnt, 1u)] = order_key(val[e]);
    }
    __syncthreads();
    const unsigned n_list = s_cnt;
    uint32_t tau;
    if (n_list <= kRankMax && n_list <= (unsigned)THREADS) {   // one thread per member
        // A short list is finished by ranking: member t is the answer when fewer than `need` members are above it and
        // at least `need` are not below it.  (Sharing a member among several threads, so that lists up to THREADS
        // members rank too, was measured slower: short lists are the rule and the extra bookkeeping hits them all.)
        if ((unsigned)tid < n_list) {
            const uint32_t kt = s_list[tid];
            unsigned gt = 0, eq = 0;
            for (unsigned u = 0; u < n_list; ++u) {
                const uint32_t v = s_list[u];
                gt += v > kt;
                eq += v == kt;
            }
            if (gt < need && need <= gt + eq) { s_prefix = kt; s_need = need - gt; s_eq = eq; }   // equal members write the same
        }
        __syncthreads();
        tau = s_prefix;
        need = s_need;
    } else {
        tau = select_on_list<THREADS>(s_list, n_list, need, hist, &s_prefix, &s_need, tid, lane, warp);
        need = s_need;
        if (tid == 0) s_eq = hist[tau & 255u];   // the last round's histogram: members equal to tau in all 32 bits
        __syncthreads();
    }
    const unsigned need_eq = need;   // equal keys kept, lowest indices first
    const bool all_ties = s_eq == need_eq;   // (the usual case: one candidate has the threshold value) every tie is kept
    const float tau_f = __uint_as_float((tau & 0x80000000u) ? (tau & 0x7fffffffu) : ~tau);

    // ---- ordered compaction with one block scan
    static_assert(E <= 64, "one 64-bit mask per thread");
    unsigned long long m_gt = 0ull, m_eq = 0ull;
    if (has)
#pragma unroll
    for (int e = 0; e < E; ++e) {
        if (all_ties) {   // uniform: the kept candidates are simply those >= tau
            m_gt |= (unsigned long long)ge_exact(val[e], tau_f) << e;
        } else {
            unsigned gt, eq;
            compare_exact(val[e], tau_f, gt, eq);
            m_gt |= (unsigned long long)gt << e;
            m_eq |= (unsigned long long)eq << e;
        }
    }
    const unsigned n_gt = __popcll(m_gt), n_eq = __popcll(m_eq);
    const unsigned packed = (n_gt << 16) | n_eq;   // both totals stay below 65536 (rows <= 32768)
    unsigned incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();   // s_warp was read by the scan above
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    unsigned wsum = lane < WARPS ? s_warp[lane] : 0u;
    unsigned wincl = wsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, wincl, o);
        if (lane >= o) wincl += t;
    }
    const unsigned excl = __shfl_sync(0xffffffffu, wincl - wsum, warp) + incl - packed;
    const unsigned gt_before = excl >> 16, eq_before = excl & 0xffffu;
    int *dst = staged ? s_out : out;
    {
        unsigned keep_eq = eq_before < need_eq ? min(n_eq, need_eq - eq_before) : 0u;
        unsigned long long m_keep = m_gt;
        while (keep_eq > 0) {   // rare: ties at the threshold
            const unsigned long long low = m_eq & (0ull - m_eq);
            m_keep |= low;
            m_eq ^= low;
            --keep_eq;
        }
        unsigned posn = gt_before + min(eq_before, need_eq);
        while (m_keep) {   // ascending candidate index
            const int e = __ffsll((long long)m_keep) - 1;
            m_keep &= m_keep - 1;
            dst[posn++] = j0 + e;
        }
    }
    if (staged) {
        __syncthreads();
        for (int t = tid; t < p.k; t += THREADS) out[t] = t < take ? s_out[t] : -1;
    } else {
        for (int t = take + tid; t < p.k; t += THREADS) out[t] = -1;
    }
}

template <int THREADS, int E, bool VEC>
__global__ void __launch_bounds__(THREADS, THREADS > 256 ? (THREADS == 512 && E <= 32 ? 2 : 1) : (E > 32 ? 2 : (HS2_TOPK_MINB32 * 256 / THREADS)))
k_topk_linear(const Params p, const float *__restrict__ scores, int64_t score_stride, int32_t *__restrict__ idx,
              int64_t row0, int nc_lo, int nc_hi, int64_t n_rows, int i_first)
{
    // i_first < 0: the CTAs walk the rows of the block in order.  Otherwise (positions known on the host) the grid covers
    // only the queries whose candidate count falls into this launch's class: x = query offset from i_first, y =
    // (sequence, KV head) from the block's first one; a launch then starts no CTAs that would leave at once.  A CTA
    // takes HS2_TOPK_ROWS consecutive rows, which spreads the cost of starting it.
    constexpr int R = HS2_TOPK_ROWS;
#pragma unroll 1
    for (int rr = 0; rr < R; ++rr) {
        const int64_t x = (int64_t)blockIdx.x * R + rr;
        int64_t row;
        if (i_first < 0) {
            row = row0 + x;
        } else {
            if (i_first + x >= p.Lq) break;
            row = (row0 / p.Lq + blockIdx.y) * p.Lq + i_first + x;
        }
        if (row >= row0 && row < row0 + n_rows) topk_linear_row<THREADS, E, VEC>(p, scores, score_stride, idx, row0, nc_lo, nc_hi, row);
        if (R > 1) __syncthreads();   // the next row reuses the shared arrays
    }
}

// ---- rows of up to CL x 32768 candidates: one thread-block cluster per row ------------------------
// Every CTA of the cluster keeps a 32768-candidate slice of the row in registers (read once).  Per
// radix round each CTA histograms its slice, CTA 0 adds the histograms up through distributed shared
// memory, picks the digit and publishes the decision; after the first round the threshold bin's
// members are appended (remote shared-memory atomics) to a list in CTA 0, which finishes the search
// alone.  The ordered compaction needs the totals of the lower-ranked CTAs, also read through DSMEM.
template <int CL, bool VEC>
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(512, 1)
k_topk_cluster(const Params p, const float *__restrict__ scores, int64_t score_stride, int32_t *__restrict__ idx,
               int64_t row0, int nc_lo, int nc_hi)
{
    namespace cg = cooperative_groups;
    constexpr int THREADS = 512, E = 64, WARPS = THREADS / 32, SLICE = THREADS * E;
    __shared__ unsigned hist[256];
    __shared__ unsigned s_sum[256];
    __shared__ unsigned s_warp[WARPS];
    __shared__ unsigned s_min[WARPS], s_max[WARPS];
    __shared__ unsigned s_mm[2];      // this CTA's min / max key
    __shared__ unsigned s_tot[2];     // this CTA's number of keys above / equal to the threshold
    __shared__ unsigned s_dec[3];     // CTA 0 publishes: digit, remaining need, size of the chosen bin
    __shared__ unsigned s_prefix, s_need, s_cnt;
    __shared__ uint32_t s_list[kListCap];

    cg::cluster_group cluster = cg::this_cluster();
    const unsigned rank = cluster.block_rank();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row = row0 + blockIdx.x / CL;   // (b, g, i), i fastest
    const int i = (int)(row % p.Lq);
    const int b = (int)(row / ((int64_t)p.Lq * p.Hkv));
    const int kvl = kvlen_of(p, b);
    const int pos = pos_of(p, b, i);
    const int nc = max(0, min(pos - p.w + 1, kvl));
    if (nc <= nc_lo || nc > nc_hi) return;   // this row belongs to another variant's launch
    const int take = min(p.k, nc);
    int32_t *out = idx + row * p.k;
    const float *srow = scores + (int64_t)(blockIdx.x / CL) * score_stride;

    if (take == nc) {   // the same branch in every CTA of the cluster; no remote access on this path
        for (int t = rank * THREADS + tid; t < p.k; t += CL * THREADS) out[t] = t < nc ? t : -1;
        return;
    }
    const int j0 = rank * SLICE + tid * E;
    uint32_t key[E];
    unsigned kmin = 0xffffffffu, kmax = 0u;
    // the slice comes in through shared memory, as in the register kernels: coalesced 16-byte copies, chunk c of the
    // slice to slot c + c / 16, each thread reading its own 16 chunks at a pitch of 17 slots
    extern __shared__ __align__(16) float s_cl_stage[];
    constexpr bool kStaged = HS2_TOPK_STAGE && VEC;
    if (kStaged) {
#pragma unroll
        for (int it = 0; it < E / 4; ++it) {
            const int c = it * THREADS + tid;
            const int jg = (int)rank * SLICE + 4 * c;
            if (jg + 4 <= nc) topk_cp_async16(s_cl_stage + (c + c / (E / 4)) * 4, srow + jg);
        }
        topk_cp_async_wait_all();
        __syncthreads();
    }
#pragma unroll
    for (int e4 = 0; e4 < E; e4 += 4) {
        if (VEC && j0 + e4 + 4 <= nc) {
            const float4 v = kStaged ? *reinterpret_cast<const float4 *>(s_cl_stage + ((E / 4 + 1) * tid + (e4 >> 2)) * 4)
                                     : __ldg(reinterpret_cast<const float4 *>(srow + j0 + e4));
            key[e4] = order_key(v.x); key[e4 + 1] = order_key(v.y); key[e4 + 2] = order_key(v.z); key[e4 + 3] = order_key(v.w);
        } else {
#pragma unroll
            for (int e = e4; e < e4 + 4; ++e) key[e] = j0 + e < nc ? order_key(srow[j0 + e]) : 0u;
        }
#pragma unroll
        for (int e = e4; e < e4 + 4; ++e)
            if (j0 + e < nc) { kmin = min(kmin, key[e]); kmax = max(kmax, key[e]); }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
        kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    if (lane == 0) { s_min[warp] = kmin; s_max[warp] = kmax; }
    __syncthreads();
    if (tid == 0) {
        unsigned a = 0xffffffffu, c = 0u;
        for (int w = 0; w < WARPS; ++w) { a = min(a, s_min[w]); c = max(c, s_max[w]); }
        s_mm[0] = a; s_mm[1] = c;
    }
    cluster.sync();
    kmin = 0xffffffffu; kmax = 0u;
#pragma unroll
    for (int r = 0; r < CL; ++r) {
        const unsigned *mm = cluster.map_shared_rank(s_mm, r);
        kmin = min(kmin, mm[0]); kmax = max(kmax, mm[1]);
    }

    int hi = 32 - __clz(kmin ^ kmax);
    unsigned prefix = hi >= 32 ? 0u : (kmax >> hi);
    unsigned need = (unsigned)take;
    unsigned *cnt0 = cluster.map_shared_rank(&s_cnt, 0);
    uint32_t *list0 = cluster.map_shared_rank(s_list, 0);
    const unsigned *dec0 = cluster.map_shared_rank(s_dec, 0);
    // Rounds on the register-resident slices (two cluster barriers each) until the threshold bin is small
    // enough for the shared list; CTA 0 then finishes alone with CTA-local barriers only.
    while (hi > 0) {
        const int w = min(8, hi), shift = hi - w;
        const unsigned dmask = (1u << w) - 1u;
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const bool live = (j0 + e < nc) && (hi >= 32 || (key[e] >> hi) == prefix);
            if (live) atomicAdd(&hist[(key[e] >> shift) & dmask], 1u);
        }
        cluster.sync();   // every CTA's histogram is complete
        if (rank == 0) {
            if (tid < 256) {
                unsigned tsum = hist[tid];
#pragma unroll
                for (int r = 1; r < CL; ++r) tsum += cluster.map_shared_rank(hist, r)[tid];
                s_sum[tid] = tsum;
            }
            __syncthreads();
            if (warp == 0) pick_digit(s_sum, prefix, need, lane, &s_prefix, &s_need);
            __syncthreads();
            if (tid == 0) {
                const unsigned digit = s_prefix & 255u;
                s_dec[0] = digit; s_dec[1] = s_need; s_dec[2] = s_sum[digit];
                s_cnt = 0;
            }
        }
        cluster.sync();   // the decision is published (and every remote histogram read is over)
        const unsigned digit = dec0[0], in_bin = dec0[2];
        need = dec0[1];
        prefix = (hi >= 32 ? 0u : (prefix << w)) | digit;
        hi = shift;
        if (hi > 0 && in_bin <= kListCap) {   // uniform over the cluster
#pragma unroll
            for (int e = 0; e < E; ++e)
                if (j0 + e < nc && (key[e] >> hi) == prefix) {
                    const unsigned slot = atomicAdd(cnt0, 1u);
                    if (slot < kListCap) list0[slot] = key[e];
                }
            cluster.sync();   // the list is complete
            if (rank == 0) {
                const unsigned n_list = min(s_cnt, kListCap);
                while (hi > 0) {
                    const int w2 = min(8, hi), shift2 = hi - w2;
                    const unsigned dmask2 = (1u << w2) - 1u;
                    if (tid < 256) hist[tid] = 0;
                    __syncthreads();
                    for (unsigned t = tid; t < n_list; t += THREADS) {
                        const uint32_t kk = s_list[t];
                        if ((kk >> hi) == prefix) atomicAdd(&hist[(kk >> shift2) & dmask2], 1u);
                    }
                    __syncthreads();
                    if (warp == 0) pick_digit(hist, prefix, need, lane, &s_prefix, &s_need);
                    __syncthreads();
                    prefix = (prefix << w2) | (s_prefix & 255u);
                    need = s_need;
                    hi = shift2;
                    __syncthreads();   // s_prefix / hist are reused by the next round
                }
                if (tid == 0) { s_dec[0] = prefix; s_dec[1] = need; }
            }
            cluster.sync();   // the final threshold is published
            prefix = dec0[0];
            need = dec0[1];
            hi = 0;
        }
        // CTA 0 overwrites s_dec only after a later cluster.sync, when every CTA has read it
    }
    const uint32_t tau = prefix;
    const unsigned need_eq = need;

    // ---- ordered compaction: block scan inside the CTA, totals of the lower-ranked CTAs through DSMEM
    unsigned n_gt = 0, n_eq = 0;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const bool ok = j0 + e < nc;
        n_gt += ok && key[e] > tau;
        n_eq += ok && key[e] == tau;
    }
    const unsigned packed = (n_gt << 16) | n_eq;   // per-CTA totals stay below 65536
    unsigned incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    unsigned wsum = lane < WARPS ? s_warp[lane] : 0u;
    unsigned wincl = wsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, wincl, o);
        if (lane >= o) wincl += t;
    }
    const unsigned excl = __shfl_sync(0xffffffffu, wincl - wsum, warp) + incl - packed;
    const unsigned cta_total = __shfl_sync(0xffffffffu, wincl, WARPS - 1);
    if (tid == 0) { s_tot[0] = cta_total >> 16; s_tot[1] = cta_total & 0xffffu; }
    cluster.sync();
    unsigned gt_before = excl >> 16, eq_before = excl & 0xffffu;
    for (unsigned r = 0; r < rank; ++r) {
        const unsigned *tot = cluster.map_shared_rank(s_tot, r);
        gt_before += tot[0]; eq_before += tot[1];
    }
#pragma unroll
    for (int e = 0; e < E; ++e) {
        if (j0 + e >= nc) continue;
        if (key[e] > tau) {
            out[gt_before + min(eq_before, need_eq)] = j0 + e;
            ++gt_before;
        } else if (key[e] == tau) {
            if (eq_before < need_eq) out[gt_before + eq_before] = j0 + e;
            ++eq_before;
        }
    }
    if (rank == 0)
        for (int t = take + tid; t < p.k; t += THREADS) out[t] = -1;
    cluster.sync();   // nobody leaves while its shared memory may still be read by a neighbour
}

// ---- longer rows: re-read from memory for every pass -------------------------------------------
// THREADS threads per row, kItems consecutive candidates per thread per step.
template <int THREADS, int ITEMS, bool CACHED, bool VEC>
__global__ void __launch_bounds__(THREADS)
k_topk(const Params p, const float *__restrict__ scores, int64_t score_stride, int32_t *__restrict__ idx,
       int64_t row0, int nc_lo, int nc_hi)
{
    constexpr int WARPS = THREADS / 32;
    constexpr int CHUNK = THREADS * kItems;           // candidates per step
    constexpr int STEPS = ITEMS / kItems;             // steps held in registers (CACHED)
    __shared__ unsigned hist[256];
    __shared__ unsigned s_warp[WARPS];
    __shared__ unsigned s_prefix, s_need;
    __shared__ unsigned s_run_gt, s_run_eq;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row = row0 + blockIdx.x;   // (b, g, i), i fastest
    const int i = (int)(row % p.Lq);
    const int b = (int)(row / ((int64_t)p.Lq * p.Hkv));
    const int kvl = kvlen_of(p, b);
    const int pos = pos_of(p, b, i);
    const int nc = max(0, min(pos - p.w + 1, kvl));   // candidates are keys 0..nc-1
    if (nc <= nc_lo || nc > nc_hi) return;   // this row belongs to another variant's launch
    const int take = min(p.k, nc);
    int32_t *out = idx + row * p.k;
    const float *srow = scores + (int64_t)blockIdx.x * score_stride;

    if (take == nc) {   // every candidate is kept: no need to look at the scores
        for (int t = tid; t < p.k; t += THREADS) out[t] = t < nc ? t : -1;
        return;
    }
    const int nsteps = (nc + CHUNK - 1) / CHUNK;

    uint32_t ck[CACHED ? ITEMS : kItems];   // cached keys (CACHED) / scratch
    if (CACHED) {
#pragma unroll
        for (int st = 0; st < STEPS; ++st) {
            if (st < nsteps) {
                uint32_t key[kItems];
                bool ok[kItems];
                load_keys<VEC>(srow, st * CHUNK + tid * kItems, nc, key, ok);
#pragma unroll
                for (int e = 0; e < kItems; ++e) ck[st * kItems + e] = key[e];
            }
        }
    }
    auto get = [&](int st, uint32_t (&key)[kItems], bool (&ok)[kItems]) {
        if (CACHED) {
#pragma unroll
            for (int s2 = 0; s2 < STEPS; ++s2)
                if (s2 == st) {
#pragma unroll
                    for (int e = 0; e < kItems; ++e) {
                        key[e] = ck[s2 * kItems + e];
                        ok[e] = st * CHUNK + tid * kItems + e < nc;
                    }
                }
        } else {
            load_keys<VEC>(srow, st * CHUNK + tid * kItems, nc, key, ok);
        }
    };

    // ---- radix select: value of the take-th largest key
    unsigned prefix = 0, need = (unsigned)take;
    for (int round = 0; round < 4; ++round) {
        const int shift = 24 - 8 * round;
        if (tid < 256) hist[tid] = 0;
        if (THREADS < 256) for (int t = tid + THREADS; t < 256; t += THREADS) hist[t] = 0;
        __syncthreads();
#pragma unroll
        for (int st = 0; st < (CACHED ? STEPS : 1); ++st) {
            for (int sr = CACHED ? st : 0; sr < (CACHED ? min(st + 1, nsteps) : nsteps); ++sr) {
                uint32_t key[kItems];
                bool ok[kItems];
                get(sr, key, ok);
#pragma unroll
                for (int e = 0; e < kItems; ++e) {
                    const bool live = ok[e] && (round == 0 || (key[e] >> (shift + 8)) == prefix);
                    const unsigned digit = live ? ((key[e] >> shift) & 255u) : 256u;
                    const unsigned peers = __match_any_sync(0xffffffffu, digit);   // one atomic per distinct digit per warp
                    if (live && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
                }
            }
        }
        __syncthreads();
        if (warp == 0) pick_digit(hist, prefix, need, lane, &s_prefix, &s_need);
        __syncthreads();
        prefix = s_prefix;
        need = s_need;
    }
    const uint32_t tau = prefix;      // key of the take-th largest candidate
    const unsigned need_eq = need;    // how many candidates equal to tau are kept (lowest indices first)

    // ---- ordered compaction: kept = key > tau, or key == tau and fewer than need_eq equal keys before it
    if (tid == 0) { s_run_gt = 0; s_run_eq = 0; }
    __syncthreads();
#pragma unroll
    for (int st = 0; st < (CACHED ? STEPS : 1); ++st) {
        for (int sr = CACHED ? st : 0; sr < (CACHED ? min(st + 1, nsteps) : nsteps); ++sr) {
            uint32_t key[kItems];
            bool ok[kItems];
            const int j0 = sr * CHUNK + tid * kItems;
            get(sr, key, ok);
            unsigned n_gt = 0, n_eq = 0;
#pragma unroll
            for (int e = 0; e < kItems; ++e) {
                n_gt += ok[e] && key[e] > tau;
                n_eq += ok[e] && key[e] == tau;
            }
            // exclusive scan of (gt, eq) over the block in thread order; both counts fit 16 bits per step
            const unsigned packed = (n_gt << 16) | n_eq;
            unsigned incl = packed;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            if (lane == 31) s_warp[warp] = incl;
            __syncthreads();
            const unsigned run_gt = s_run_gt, run_eq = s_run_eq;
            unsigned wsum = lane < WARPS ? s_warp[lane] : 0u;   // every warp scans the warp totals itself
            unsigned wincl = wsum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned t = __shfl_up_sync(0xffffffffu, wincl, o);
                if (lane >= o) wincl += t;
            }
            const unsigned warp_excl = __shfl_sync(0xffffffffu, wincl - wsum, warp);
            const unsigned total = __shfl_sync(0xffffffffu, wincl, WARPS - 1);
            const unsigned excl = warp_excl + incl - packed;
            unsigned gt_before = run_gt + (excl >> 16), eq_before = run_eq + (excl & 0xffffu);
#pragma unroll
            for (int e = 0; e < kItems; ++e) {
                if (!ok[e]) continue;
                if (key[e] > tau) {
                    out[gt_before + min(eq_before, need_eq)] = j0 + e;
                    ++gt_before;
                } else if (key[e] == tau) {
                    if (eq_before < need_eq) out[gt_before + eq_before] = j0 + e;
                    ++eq_before;
                }
            }
            __syncthreads();   // everyone has read s_warp and the running totals
            if (tid == 0) { s_run_gt = run_gt + (total >> 16); s_run_eq = run_eq + (total & 0xffffu); }
        }
    }
    for (int t = take + tid; t < p.k; t += THREADS) out[t] = -1;
}

}  // namespace

// Variants by the number of candidates of a row: (lo, hi] -> kernel.  A launch covers every row of the
// block; rows outside the variant's range leave at once, so each row is handled by exactly one launch
// and the choice is per row even when the positions live on the device.
struct TopkClass { int lo, hi; };
constexpr int kNumClasses = 9;
constexpr TopkClass kClasses[kNumClasses] = {{-1, 2048},      {2048, 4096},     {4096, 8192},        {8192, 16384},
                                             {16384, 32768},  {32768, 65536},   {65536, 131072},     {131072, 262144},
                                             {262144, 0x7fffffff}};

template <bool VEC>
cudaError_t launch_class(int c, const Params &p, const float *scores, int64_t score_stride, int32_t *idx, int64_t row0,
                         int64_t n_rows, cudaStream_t st)
{
    const int lo = kClasses[c].lo, hi = kClasses[c].hi;
    const unsigned n = (unsigned)n_rows;
    const size_t stage = p.k <= kStageOut ? (size_t)p.k * sizeof(int) : 0;   // the register kernels stage their output row
#ifdef HS2_TOPK_NO_CLUSTER
    if (c >= 5 && c <= 7) c = 8;   // tuning builds: long rows on the streaming kernel
#endif
    // The register kernels pay a fixed price per warp and row (rounds, scans, barriers), so a row gets no more
    // warps than its candidates fill: 32 (or 64) candidates per thread.
#if HS2_TOPK_LINEAR
    if (c <= 4) {   // register-resident rows: first round on a linear scale, the threshold bin's members in a shared list
        cudaError_t err = cudaSuccess;
        auto go = [&](auto kern, int threads, int e) -> bool {   // false: nothing was launched (err says whether that is a failure)
            // (+ one 16-byte slot per thread and the alignment of the staged row, which passes through the list's memory)
            const size_t smem = stage + (size_t)threads * e * sizeof(uint32_t) + (size_t)threads * 16 + 16;
            if (smem > 32 * 1024) {   // static shared memory counts against the 48 KB default too
                static bool attr_set[5][64] = {};   // per row class: the kernels share one function type, hence one lambda body
                int dev = 0;
                if ((err = cudaGetDevice(&dev)) != cudaSuccess) return false;
                if (!(dev >= 0 && dev < 64 && attr_set[c][dev])) {
                    if ((err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                    (int)(kStageOut * sizeof(int) + (size_t)threads * e * sizeof(uint32_t) + (size_t)threads * 16 + 16))) != cudaSuccess)
                        return false;
                    if (dev >= 0 && dev < 64) attr_set[c][dev] = true;
                }
            }
            // the queries of this class, when the candidate count is a known function of the query index
            if (!p.q_start && !p.kv_lens) {
                const int64_t base = (int64_t)p.Lk - p.Lq - p.w + 1;   // candidates of query i: clamp(base + i, 0, Lk)
                int64_t i_lo = lo < 0 ? 0 : (int64_t)lo + 1 - base, i_hi = hi >= p.Lk ? (int64_t)p.Lq - 1 : (int64_t)hi - base;
                if (i_lo < 0) i_lo = 0;
                if (i_hi > p.Lq - 1) i_hi = p.Lq - 1;
                if (i_hi < i_lo) return false;
                const int64_t n_bg = (row0 + n_rows - 1) / p.Lq - row0 / p.Lq + 1;
                if (n_bg <= 65535) {
                    kern<<<dim3((unsigned)((i_hi - i_lo + HS2_TOPK_ROWS) / HS2_TOPK_ROWS), (unsigned)n_bg), threads, smem, st>>>(
                        p, scores, score_stride, idx, row0, lo, hi, n_rows, (int)i_lo);
                    return true;
                }
            }
            kern<<<(n + HS2_TOPK_ROWS - 1) / HS2_TOPK_ROWS, threads, smem, st>>>(p, scores, score_stride, idx, row0, lo, hi, n_rows, -1);
            return true;
        };
        bool launched = false;
        switch (c) {
            case 0: launched = go(k_topk_linear<64, 32, VEC>, 64, 32); break;
            case 1: launched = go(k_topk_linear<128, 32, VEC>, 128, 32); break;
            case 2: launched = go(k_topk_linear<256, 32, VEC>, 256, 32); break;
#if HS2_TOPK_WIDE
            case 3: launched = go(k_topk_linear<512, 32, VEC>, 512, 32); break;
#else
            case 3: launched = go(k_topk_linear<256, 64, VEC>, 256, 64); break;
#endif
            default: launched = go(k_topk_linear<512, 64, VEC>, 512, 64); break;
        }
        if (launched) count_launch();
        return err;
    }
#endif
    switch (c) {
        case 0: k_topk_cached<64, 32, VEC><<<n, 64, stage, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
        case 1: k_topk_cached<128, 32, VEC><<<n, 128, stage, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
        case 2: k_topk_cached<256, 32, VEC><<<n, 256, stage, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
        case 3: k_topk_cached<256, 64, VEC><<<n, 256, stage, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
        case 4: k_topk_cached<512, 64, VEC><<<n, 512, stage, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
        case 5: case 6: case 7: {   // (dynamic shared memory: the staged slice of the row)
            const size_t smem = (HS2_TOPK_STAGE && VEC) ? cached_stage_bytes(512, 64) : 0;
            auto go = [&](auto kern, unsigned cl) -> cudaError_t {
                if (smem > 48 * 1024) {
                    static bool attr_set[3][64] = {};   // per cluster size and device ordinal
                    int dev = 0;
                    cudaError_t e = cudaGetDevice(&dev);
                    if (e != cudaSuccess) return e;
                    if (!(dev >= 0 && dev < 64 && attr_set[c - 5][dev])) {
                        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
                        if (dev >= 0 && dev < 64) attr_set[c - 5][dev] = true;
                    }
                }
                kern<<<n * cl, 512, smem, st>>>(p, scores, score_stride, idx, row0, lo, hi);
                return cudaSuccess;
            };
            const cudaError_t e = c == 5 ? go(k_topk_cluster<2, VEC>, 2u) : c == 6 ? go(k_topk_cluster<4, VEC>, 4u) : go(k_topk_cluster<8, VEC>, 8u);
            if (e != cudaSuccess) return e;   // nothing was launched: the rows of this class would stay unwritten
            break;
        }
        default: k_topk<1024, kItems, false, VEC><<<n, 1024, 0, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
    }
    count_launch();
    return cudaSuccess;
}

cudaError_t launch_topk(const Params &p, const float *scores, int64_t score_stride, int32_t *idx, int64_t row0,
                        int64_t n_rows, cudaStream_t st)
{
    if (n_rows == 0 || p.k == 0) return cudaSuccess;
    const bool vec = (score_stride % 4 == 0) && (reinterpret_cast<uintptr_t>(scores) % 16 == 0);
    // range of candidate counts that can occur in this block of rows
    int64_t nc_min = 0, nc_max = p.Lk;
    if (!p.q_start && !p.kv_lens) {
        // host-known positions: query i has clamp(Lk - Lq + i - w + 1, 0, Lk) candidates, growing with i
        const int64_t base = (int64_t)p.Lk - p.Lq - p.w + 1;
        const int64_t i_first = row0 % p.Lq, i_last = (row0 + n_rows - 1) % p.Lq;
        const bool wraps = (row0 / p.Lq) != ((row0 + n_rows - 1) / p.Lq);
        const int64_t i_lo = wraps ? 0 : i_first, i_hi = wraps ? p.Lq - 1 : i_last;
        auto clampnc = [&](int64_t v) { return v < 0 ? (int64_t)0 : (v > p.Lk ? (int64_t)p.Lk : v); };
        nc_min = clampnc(base + i_lo);
        nc_max = clampnc(base + i_hi);
    }
    for (int c = 0; c < kNumClasses; ++c) {
        if (nc_max <= kClasses[c].lo || nc_min > kClasses[c].hi) continue;   // no row of the block falls in this class
        const cudaError_t e = vec ? launch_class<true>(c, p, scores, score_stride, idx, row0, n_rows, st)
                                  : launch_class<false>(c, p, scores, score_stride, idx, row0, n_rows, st);
        if (e != cudaSuccess) return e;
    }
    return cudaGetLastError();
}


// ---- exact redo of flagged rows -------------------------------------------------------------------
// The filtered pipeline marks a row when its candidate count came out below the number to select or
// above the list capacity (the sampled threshold was off, which needs adversarially structured scores).
// Such a row is selected here from scores recomputed on the fly, pass by pass (bf16 inputs, fp32 FMAs):
// slow, but it needs no storage, no host round trip, and handles any number of rows.
namespace {

constexpr int kRedoChunk = 64;

__global__ void __launch_bounds__(256)
k_select_recompute(const Params p, const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                   const float *__restrict__ LSE, int32_t *__restrict__ idx, int64_t row0, int64_t n_rows,
                   const int *__restrict__ flag)
{
    constexpr int THREADS = 256, WARPS = 8, D = 128;
    extern __shared__ float sq[];                 // [G][128] queries, then [G] LSE
    __shared__ unsigned hist[256];
    __shared__ unsigned s_warp[WARPS];
    __shared__ unsigned s_prefix, s_need, s_run_gt, s_run_eq;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // The rows of the block are walked in chunks of kRedoChunk rows: one coalesced load and one barrier tell a CTA
    // whether any row of its chunk is flagged, so a launch that finds none (the usual case) costs a few microseconds
    // whatever the number of rows; the flagged rows of one chunk are redone one after the other.
    __shared__ int s_flagged[kRedoChunk];
    for (int64_t chunk = (int64_t)blockIdx.x * kRedoChunk; chunk < n_rows; chunk += (int64_t)gridDim.x * kRedoChunk) {
        const int mine = tid < kRedoChunk && chunk + tid < n_rows ? flag[chunk + tid] : 0;
        if (!__syncthreads_or(mine)) continue;
        if (tid < kRedoChunk) s_flagged[tid] = mine;
        __syncthreads();
        for (int r = 0; r < kRedoChunk && chunk + r < n_rows; ++r) {
            if (!s_flagged[r]) continue;   // (the same for every thread of the CTA)
            const int64_t lr = chunk + r;
            const int64_t row = row0 + lr;
            const int i = (int)(row % p.Lq);
            const int g = (int)((row / p.Lq) % p.Hkv);
            const int b = (int)(row / ((int64_t)p.Lq * p.Hkv));
            const int kvl = kvlen_of(p, b);
            const int pos = pos_of(p, b, i);
            const int nc = max(0, min(pos - p.w + 1, kvl));
            const int take = min(p.k, nc);
            int32_t *out = idx + row * p.k;
            float *slse = sq + p.G * D;
            for (int e = tid; e < p.G * D; e += THREADS)
                sq[e] = __bfloat162float(Q[b * p.qs_b + (int64_t)i * p.qs_t + (g * p.G + e / D) * p.qs_h + e % D]);
            for (int e = tid; e < p.G; e += THREADS) slse[e] = LSE[((int64_t)b * p.Hq + g * p.G + e) * p.Lq + i];
            __syncthreads();
            const __nv_bfloat16 *kb = K + b * p.ks_b + g * p.ks_h;
            auto key_of = [&](int j) -> uint32_t {   // order key of a[j] = max_h (scale <q_h, k_j> - LSE_h)
                const uint4 *kr = reinterpret_cast<const uint4 *>(kb + (int64_t)j * p.ks_t);
                float kf[D];
        #pragma unroll
                for (int c = 0; c < D / 8; ++c) {
                    const uint4 v = __ldg(kr + c);
                    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        #pragma unroll
                    for (int t = 0; t < 4; ++t) { kf[8 * c + 2 * t] = __uint_as_float(w[t] << 16); kf[8 * c + 2 * t + 1] = __uint_as_float(w[t] & 0xffff0000u); }
                }
                float best = -INFINITY;
                for (int h = 0; h < p.G; ++h) {
                    float acc = 0.f;
        #pragma unroll
                    for (int d = 0; d < D; ++d) acc = fmaf(kf[d], sq[h * D + d], acc);
                    best = fmaxf(best, fmaf(acc, p.scale, -slse[h]));
                }
                return order_key(best);
            };
            unsigned prefix = 0, need = (unsigned)take;
            for (int round = 0; round < 4; ++round) {
                const int shift = 24 - 8 * round;
                hist[tid] = 0;
                __syncthreads();
                for (int base = 0; base < nc; base += THREADS) {
                    const int j = base + tid;
                    const uint32_t kk = j < nc ? key_of(j) : 0u;
                    const bool live = j < nc && (round == 0 || (kk >> (shift + 8)) == prefix);
                    const unsigned digit = live ? ((kk >> shift) & 255u) : 256u;
                    const unsigned peers = __match_any_sync(0xffffffffu, digit);
                    if (live && lane == __ffs(peers) - 1) atomicAdd(&hist[digit], __popc(peers));
                }
                __syncthreads();
                if (warp == 0) pick_digit(hist, prefix, need, lane, &s_prefix, &s_need);
                __syncthreads();
                prefix = s_prefix;
                need = s_need;
            }
            const uint32_t tau = prefix;
            const unsigned need_eq = need;
            if (tid == 0) { s_run_gt = 0; s_run_eq = 0; }
            __syncthreads();
            for (int base = 0; base < nc; base += THREADS) {
                const int j = base + tid;
                const uint32_t kk = j < nc ? key_of(j) : 0u;
                const unsigned gt = j < nc && kk > tau, eq = j < nc && kk == tau;
                const unsigned bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
                if (lane == 0) s_warp[warp] = (__popc(bg) << 16) | __popc(be);
                __syncthreads();
                unsigned gt_before = s_run_gt, eq_before = s_run_eq, tot_gt = 0, tot_eq = 0;
        #pragma unroll
                for (int w2 = 0; w2 < WARPS; ++w2) {
                    const unsigned c = s_warp[w2];
                    if (w2 < warp) { gt_before += c >> 16; eq_before += c & 0xffffu; }
                    tot_gt += c >> 16; tot_eq += c & 0xffffu;
                }
                const unsigned lt = (1u << lane) - 1u;
                gt_before += __popc(bg & lt);
                eq_before += __popc(be & lt);
                if (gt) out[gt_before + min(eq_before, need_eq)] = j;
                else if (eq && eq_before < need_eq) out[gt_before + eq_before] = j;
                __syncthreads();
                if (tid == 0) { s_run_gt += tot_gt; s_run_eq += tot_eq; }
                __syncthreads();
            }
            for (int t = take + tid; t < p.k; t += THREADS) out[t] = -1;
                __syncthreads();   // the next row reuses the shared arrays
        }
        __syncthreads();   // s_flagged is rewritten for the next chunk
    }
}

}  // namespace

int filter_sample_width(const Params &p, int samp)
{
    return ((p.Lk + 128 * samp - 1) / (128 * samp)) * 128;   // sampled scores per row, padded to whole tiles
}

// thresholds tau_key[row] from the sampled strips (row stride `stride` floats); clears flag[row]
// ---- block-level selection (the variant the paper ablates against: Section 5, Ablation 1) --------------------------
// One warp per row.  The row's candidates 0..n-1 are cut into aligned blocks of p.blk keys (the last one may be
// partial); a block's score is the maximum over its candidate keys; the k/blk best blocks (ties: lower block first)
// are kept and their candidate keys written in ascending order.  The row is read once, coalesced; the block maxima
// live in the warp's shared memory; the selection is k/blk rounds of a warp-wide argmax.
constexpr int kBlkWarps = 8;

__global__ void __launch_bounds__(kBlkWarps * 32)
k_block_select(const Params p, const float *__restrict__ scores, int64_t score_stride, int32_t *__restrict__ idx, int64_t row0,
               int64_t n_rows, int nb_max)
{
    extern __shared__ uint32_t s_blk[];   // [kBlkWarps][nb_max] block maxima as order-preserving keys; [kBlkWarps][k/blk] winners
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t lr = (int64_t)blockIdx.x * kBlkWarps + warp;
    if (lr >= n_rows) return;
    const int64_t row = row0 + lr;
    const int i = (int)(row % p.Lq);
    const int b = (int)(row / ((int64_t)p.Lq * p.Hkv));
    const int kvl = kvlen_of(p, b);
    const int pos = pos_of(p, b, i);
    const int n = max(0, min(pos - p.w + 1, kvl));
    const int B = p.blk, kb = p.k / B;
    const int nb = (n + B - 1) / B;
    int32_t *out = idx + row * p.k;
    uint32_t *bk = s_blk + (size_t)warp * nb_max;
    int *win = reinterpret_cast<int *>(s_blk + (size_t)kBlkWarps * nb_max) + warp * kb;
    const float *srow = scores + lr * score_stride;
    const int take = min(kb, nb);
    if (take < nb) {
        // block maxima: lane l folds keys l, l + 32, ... of a block, then a warp maximum.  0 marks "already taken",
        // and no real score maps to key 0 (the key of the NaN with all bits set)
        for (int m = 0; m < nb; ++m) {
            uint32_t best = 1u;
            const int hi = min(n, (m + 1) * B);
            for (int j = m * B + lane; j < hi; j += 32) best = max(best, max(order_key(srow[j]), 1u));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
            if (lane == 0) bk[m] = best;
        }
        __syncwarp();
        for (int r = 0; r < take; ++r) {
            // argmax with ties to the lower block: compare (key, ~block)
            unsigned long long best = 0ull;
            for (int m = lane; m < nb; m += 32) {
                const unsigned long long c = ((unsigned long long)bk[m] << 32) | (uint32_t)(~m);
                if (bk[m] != 0u && c > best) best = c;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const unsigned long long t = __shfl_xor_sync(0xffffffffu, best, o);
                best = t > best ? t : best;
            }
            const int m = (int)~(uint32_t)best;
            if (lane == 0) { win[r] = m; bk[m] = 0u; }
            __syncwarp();
        }
        // ascending block order: rank of each winner among the winners (take <= k / blk is small)
        int mine[2] = {-1, -1}, rank[2] = {0, 0};
        for (int u = 0; u < 2; ++u) {
            const int r = lane + 32 * u;
            if (r < take) {
                mine[u] = win[r];
                for (int q = 0; q < take; ++q) rank[u] += win[q] < mine[u];
            }
        }
        __syncwarp();
        if (take <= 64) {
            for (int u = 0; u < 2; ++u)
                if (mine[u] >= 0) win[rank[u]] = mine[u];
        } else if (lane == 0) {   // many blocks per row: a plain insertion sort by one lane
            for (int a = 1; a < take; ++a) {
                const int v = win[a];
                int c = a - 1;
                while (c >= 0 && win[c] > v) { win[c + 1] = win[c]; --c; }
                win[c + 1] = v;
            }
        }
        __syncwarp();
    }
    // emit the candidate keys of the kept blocks, ascending; a partial last block gives fewer than B keys
    int written = 0;
    for (int r = 0; r < take; ++r) {
        const int m = take < nb ? win[r] : r;
        const int lo = m * B, hi = min(n, lo + B);
        for (int j = lo + lane; j < hi; j += 32) out[written + (j - lo)] = j;
        written += hi - lo;
    }
    for (int t = written + lane; t < p.k; t += 32) out[t] = -1;
}

cudaError_t launch_block_select(const Params &p, const float *scores, int64_t score_stride, int32_t *idx, int64_t row0,
                                int64_t n_rows, cudaStream_t st)
{
    if (n_rows <= 0 || p.k <= 0) return cudaSuccess;
    const int nb_max = (p.Lk + p.blk - 1) / p.blk;
    const size_t smem = (size_t)kBlkWarps * (nb_max + p.k / p.blk) * sizeof(uint32_t);
    if (smem > 200 * 1024) return cudaErrorNotSupported;
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !done[dev]) {
        if ((e = cudaFuncSetAttribute(k_block_select, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)) != cudaSuccess) return e;
        done[dev] = true;
    }
    const int64_t grid = (n_rows + kBlkWarps - 1) / kBlkWarps;
    if (grid > 0x7fffffffLL) return cudaErrorNotSupported;
    k_block_select<<<(unsigned)grid, kBlkWarps * 32, smem, st>>>(p, scores, score_stride, idx, row0, n_rows, nb_max);
    count_launch();
    return cudaGetLastError();
}

// ---- the two selects of the filtered path --------------------------------------------------------------------------
// Both want one thing first: the value at a given rank from the top of an unordered set (the threshold from a row's
// sampled scores; the k-th best of a row's candidate list).  Order does not matter for that, so the values are read
// strided - thread t takes entries t, t + THREADS, ... - which is coalesced without any staging and gives every
// thread the same share whatever the set's size.  The rank is found as in k_topk_linear: one round of bins on a
// linear scale between the set's smallest and largest value, then an exact ranking of the threshold bin's members.
namespace {

constexpr int kCandList = 4096;   // words of the candidate select's list (later its staged output row)

struct RankOut {
    uint32_t tau;       // order key of the value at rank `take` from the top
    unsigned need_eq;   // how many of the entries equal to it belong to the top `take`
    unsigned n_eq;      // how many entries equal it
    bool ok;            // false: the threshold bin has more members than the list holds (nothing else is valid then)
};

// val[0 .. nv) are this thread's live entries; `take` >= 1 and at most the number of live entries of the CTA.
// hist: 4 * THREADS words; s_list: list_cap words; every thread of the CTA must call.
// BOTTOM: the wanted rank lies in the lower part of the set and the set thins out towards the top (a candidate list:
// everything above a threshold, most of it to be kept).  Bins between the smallest and the largest value would then
// put the dense lower part, where the answer is, into a few bins; instead the bins span twice the distance from the
// smallest value to the mean (n_live entries in all) and the last bin takes everything above.  Any monotone map to
// bins is exact; the choice only decides how many members the threshold bin has.
template <int THREADS, int E, bool BOTTOM>
__device__ __forceinline__ RankOut rank_from_top(const float (&val)[E], int nv, unsigned take, unsigned n_live, unsigned *hist,
                                                 uint32_t *s_list, unsigned list_cap, float *s_lo, float *s_hi, unsigned *s_warp,
                                                 unsigned *s_misc, int tid, int lane, int warp)
{
    constexpr int WARPS = THREADS / 32;
    constexpr int NBT = 4, NB = NBT * THREADS;
    unsigned &s_prefix = s_misc[0], &s_need = s_misc[1], &s_cnt = s_misc[2], &s_bin = s_misc[3], &s_eq = s_misc[4];
    const int nvw = __reduce_max_sync(0xffffffffu, nv);   // the unrolled per-entry loops stop at the warp's longest thread
    float vmin = INFINITY, vmax = -INFINITY;   // with BOTTOM, vmax carries the sum instead
    if (BOTTOM) vmax = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        if (e >= nvw) break;
        if (e < nv) { vmin = fminf(vmin, val[e]); vmax = BOTTOM ? vmax + val[e] : fmaxf(vmax, val[e]); }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        vmin = fminf(vmin, __shfl_xor_sync(0xffffffffu, vmin, o));
        const float t = __shfl_xor_sync(0xffffffffu, vmax, o);
        vmax = BOTTOM ? vmax + t : fmaxf(vmax, t);
    }
    __syncthreads();   // the shared arrays may still be in use by an earlier phase of the caller
    if (lane == 0) { s_lo[warp] = vmin; s_hi[warp] = vmax; }
#pragma unroll
    for (int t = 0; t < NBT; ++t) hist[t * THREADS + tid] = 0u;
    if (tid == 0) s_cnt = 0u;
    __syncthreads();
    vmin = s_lo[0]; vmax = s_hi[0];
#pragma unroll
    for (int w = 1; w < WARPS; ++w) { vmin = fminf(vmin, s_lo[w]); vmax = BOTTOM ? vmax + s_hi[w] : fmaxf(vmax, s_hi[w]); }
    const float range = BOTTOM ? 2.f * (vmax / (float)n_live - vmin) : vmax - vmin;
    const bool flat = !(range > 0.f) || !(range < 3.0e38f);
    const float c = flat ? 0.f : (float)NB / range;
    const float d = flat ? 0.f : -vmin * c;
    auto bin_of = [&](float v) { return min(__float2uint_rd(__fmaf_rn(v, c, d)), (unsigned)(NB - 1)); };
#pragma unroll
    for (int e = 0; e < E; ++e) {
        if (e >= nvw) break;
        if (e < nv) atomicAdd(&hist[bin_of(val[e])], 1u);
    }
    __syncthreads();
    unsigned mine = 0;
#pragma unroll
    for (int e = 0; e < NBT; ++e) mine += hist[NB - 1 - NBT * tid - e];
    unsigned total;
    const unsigned before = block_excl_scan<WARPS>(mine, s_warp, lane, warp, &total);
    if (before < take && take <= before + mine) {
        unsigned cum = before;
#pragma unroll
        for (int e = 0; e < NBT; ++e) {
            const unsigned cnt = hist[NB - 1 - NBT * tid - e];
            if (cum < take && take <= cum + cnt) { s_bin = NB - 1 - NBT * tid - e; s_need = take - cum; }
            cum += cnt;
        }
    }
    __syncthreads();
    const unsigned tbin = s_bin;
    unsigned need = s_need;
    const float x_lo = tbin == 0u ? -INFINITY : (float)tbin;
    const float x_hi = tbin == (unsigned)(NB - 1) ? __uint_as_float(0x7fc00000u) : (float)(tbin + 1u);
#pragma unroll
    for (int e = 0; e < E; ++e) {
        if (e >= nvw) break;
        if (e < nv) {
            const float x = __fmaf_rn(val[e], c, d);
            if (!(x < x_lo) && !(x >= x_hi)) {
                const unsigned slot = atomicAdd(&s_cnt, 1u);
                if (slot < list_cap) s_list[slot] = order_key(val[e]);
            }
        }
    }
    __syncthreads();
    const unsigned n_list = s_cnt;
    RankOut r;
    r.ok = n_list <= list_cap;
    if (!r.ok) {
        r.tau = 0u; r.need_eq = 0u; r.n_eq = 0u;
        return r;
    }
    if (n_list <= kRankMax && n_list <= (unsigned)THREADS) {
        if ((unsigned)tid < n_list) {
            const uint32_t kt = s_list[tid];
            unsigned gt = 0, eq = 0;
            for (unsigned u = 0; u < n_list; ++u) {
                const uint32_t v = s_list[u];
                gt += v > kt;
                eq += v == kt;
            }
            if (gt < need && need <= gt + eq) { s_prefix = kt; s_need = need - gt; s_eq = eq; }
        }
        __syncthreads();
        r.tau = s_prefix;
    } else {
        r.tau = select_on_list<THREADS>(s_list, n_list, need, hist, &s_prefix, &s_need, tid, lane, warp);
        if (tid == 0) s_eq = hist[r.tau & 255u];   // the last round's histogram: members equal to tau in all 32 bits
        __syncthreads();
    }
    r.need_eq = s_need;
    r.n_eq = s_eq;
    return r;
}

// Threshold of a row from its sampled scores: the value at rank sample_rank() of the sample (see there).
// One CTA per row; a launch takes the rows whose sample size lies in (ns_lo, ns_hi].
template <int THREADS, int E>
__global__ void __launch_bounds__(THREADS, E >= 64 ? 1 : (THREADS > 256 ? 2 : (E > 16 ? 3 : 1024 / THREADS)))
k_sample_tau(const Params p, const float *__restrict__ sample, int64_t stride, int64_t row0, int ns_lo, int ns_hi, int samp,
             int cap, uint32_t *__restrict__ tau_key, int *__restrict__ flag)
{
    constexpr int WARPS = THREADS / 32;
    __shared__ unsigned hist[4 * THREADS];
    __shared__ unsigned s_warp[WARPS];
    __shared__ float s_lo[WARPS], s_hi[WARPS];
    __shared__ unsigned s_misc[8];
    extern __shared__ uint32_t s_tau_list[];   // THREADS * E keys
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row = row0 + blockIdx.x;
    const int i = (int)(row % p.Lq);
    const int b = (int)(row / ((int64_t)p.Lq * p.Hkv));
    const int n_keys = max(0, min(pos_of(p, b, i) - p.w + 1, kvlen_of(p, b)));
    const int k_row = min(p.k, n_keys);
    const int nc = sample_size(n_keys, samp);
    if (nc <= ns_lo || nc > ns_hi) return;   // another class's row
    const int take = n_keys > 0 ? min(nc, sample_rank(k_row, n_keys, nc)) : 0;
    if (tid == 0) flag[blockIdx.x] = 0;
    if (n_keys <= cap || take <= 0) {   // short row: every key is a candidate
        if (tid == 0) tau_key[blockIdx.x] = 0u;
        return;
    }
    const float *srow = sample + (int64_t)blockIdx.x * stride;
    float val[E];
    const int nv = nc > tid ? min(E, (nc - tid + THREADS - 1) / THREADS) : 0;
#pragma unroll
    for (int e = 0; e < E; ++e) val[e] = e < nv ? __ldg(srow + tid + THREADS * e) : 0.f;
    const RankOut r = rank_from_top<THREADS, E, false>(val, nv, (unsigned)take, (unsigned)nc, hist, s_tau_list, (unsigned)(THREADS * E), s_lo,
                                                       s_hi, s_warp, s_misc, tid, lane, warp);
    if (tid == 0) tau_key[blockIdx.x] = r.tau;
}

// Final selection of a row from its candidate list (four sub-lists, see the score sweep): the k best by (score
// descending, key ascending), written in ascending key order.  Thread groups of THREADS / 4 take one sub-list each,
// strided.  The kept keys are marked in a bitmap over the row's keys, which is then read out in order.
// Rows whose list is unusable (a sub-list overflowed or was abandoned, fewer candidates than wanted) are flagged for
// the exact redo.
template <int THREADS, int E>
__global__ void __launch_bounds__(THREADS, THREADS > 256 ? 1 : (E > 16 ? 3 : 1024 / THREADS))
k_cand_select(const Params p, const int2 *__restrict__ cand, const int *__restrict__ count,
              int cap, int32_t *__restrict__ idx, int64_t row0, int *__restrict__ flag)
{
    constexpr int WARPS = THREADS / 32, TG = THREADS / 4;
    __shared__ unsigned hist[4 * THREADS];
    __shared__ unsigned s_warp[WARPS];
    __shared__ float s_lo[WARPS], s_hi[WARPS];
    __shared__ unsigned s_misc[8];
    extern __shared__ __align__(16) unsigned char s_cs_dyn[];   // [bitmap over the row's keys][list / staged output][key indices]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row = row0 + blockIdx.x;
    const int i = (int)(row % p.Lq);
    const int b = (int)(row / ((int64_t)p.Lq * p.Hkv));
    const int n_keys = max(0, min(pos_of(p, b, i) - p.w + 1, kvlen_of(p, b)));
    const int k_row = min(p.k, n_keys);
    int32_t *out = idx + row * p.k;
    if (k_row == n_keys) {   // every candidate is kept: no need to look at the scores
        for (int t = tid; t < p.k; t += THREADS) out[t] = t < n_keys ? t : -1;
        return;
    }
    const int capq = cap >> 2;
    int total = 0, mine_cnt = 0;
    bool bad = false;
#pragma unroll
    for (int sub = 0; sub < 4; ++sub) {
        const int c = count[(int64_t)blockIdx.x * 4 + sub];
        bad |= c < 0 || c > capq;
        total += c;
        if (tid / TG == sub) mine_cnt = c;
    }
    if (bad || total < k_row) {   // the threshold was off (or the sweep gave up): redo this row exactly
        if (tid == 0) flag[blockIdx.x] = 1;
        return;
    }
    unsigned *bitmap = reinterpret_cast<unsigned *>(s_cs_dyn);
    uint32_t *s_list = reinterpret_cast<uint32_t *>(s_cs_dyn + cached_bitmap_bytes(p.Lk));   // kCandList words
    int32_t *s_pay = reinterpret_cast<int32_t *>(s_list + kCandList);                         // THREADS * E key indices
    const int l = tid % TG;
    const int64_t base = (int64_t)blockIdx.x * cap + (tid / TG) * capq + l;   // this thread's entries: base + TG * e
    const int nv = mine_cnt > l ? min(E, (mine_cnt - l + TG - 1) / TG) : 0;
    const int nvw = __reduce_max_sync(0xffffffffu, nv);   // the unrolled per-entry loops stop at the warp's longest thread
    float val[E];
    // a record is (score, key): the score stays in a register, the key waits in shared memory until the threshold is
    // known (each thread reads back only what it stored itself)
#pragma unroll
    for (int e = 0; e < E; ++e) {
        val[e] = 0.f;
        if (e < nv) {
            const int2 rec = __ldg(cand + base + TG * e);
            val[e] = __int_as_float(rec.x) * p.scale;   // the sweep stores the accumulator's value: the score is that times scale
            s_pay[e * THREADS + tid] = rec.y;
        }
    }
    const int nwords = (n_keys + 31) >> 5;
    for (int wd = tid; wd < nwords; wd += THREADS) bitmap[wd] = 0u;   // (rank_from_top's barriers order this before the marking)
    const RankOut r = rank_from_top<THREADS, E, true>(val, nv, (unsigned)k_row, (unsigned)total, hist, s_list, (unsigned)kCandList, s_lo,
                                                      s_hi, s_warp, s_misc, tid, lane, warp);
    if (!r.ok || r.n_eq > (unsigned)kCandList) {   // thousands of candidates within one bin of the threshold: the exact redo takes the row
        if (tid == 0) flag[blockIdx.x] = 1;
        return;
    }
    const float tau_f = __uint_as_float((r.tau & 0x80000000u) ? (r.tau & 0x7fffffffu) : ~r.tau);
    uint32_t jmin = 0u;   // of the candidates equal to the threshold, those with ~key >= jmin are kept
    if (r.n_eq > r.need_eq) {   // ties at the threshold, not all of them wanted: the lowest keys win
        __syncthreads();
        if (tid == 0) s_misc[2] = 0u;
        __syncthreads();
#pragma unroll
        for (int e = 0; e < E; ++e)
            if (e < nv && order_key(val[e]) == r.tau) s_list[atomicAdd(&s_misc[2], 1u)] = ~(uint32_t)s_pay[e * THREADS + tid];
        __syncthreads();
        jmin = select_on_list<THREADS>(s_list, r.n_eq, r.need_eq, hist, &s_misc[0], &s_misc[1], tid, lane, warp);
    }
    // mark the kept keys (the comparison must see denormal scores as they are)
#pragma unroll
    for (int e = 0; e < E; ++e) {
        if (e >= nvw) break;
        if (e < nv && ge_exact(val[e], tau_f)) {
            const uint32_t j = (uint32_t)s_pay[e * THREADS + tid];
            // (the sweep only writes keys below n_keys; the range test keeps a damaged list from writing outside the bitmap)
            if (j < (uint32_t)n_keys && (jmin == 0u || ~j >= jmin || order_key(val[e]) != r.tau)) atomicOr(&bitmap[j >> 5], 1u << (j & 31u));
        }
    }
    __syncthreads();
    // Read the bitmap out in ascending key order.  A warp takes a contiguous run of words, its lanes consecutive words
    // (no bank conflicts); the position of a word's first kept key is the warp's base plus a shuffle scan of the counts.
    const int per_warp = ((nwords + WARPS - 1) / WARPS + 31) & ~31;
    const int wbeg = warp * per_warp;
    unsigned kept = 0;
    for (int wd = wbeg + lane; wd < min(nwords, wbeg + per_warp); wd += 32) kept += __popc(bitmap[wd]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) kept += __shfl_xor_sync(0xffffffffu, kept, o);
    __syncthreads();   // s_warp may still be read by an earlier scan
    if (lane == 0) s_warp[warp] = kept;
    __syncthreads();
    unsigned run = 0, total_sel = 0;
#pragma unroll
    for (int w = 0; w < WARPS; ++w) {
        if (w < warp) run += s_warp[w];
        total_sel += s_warp[w];
    }
    const bool staged = k_row <= kCandList;   // the list's memory is free now: the row leaves as coalesced stores
    int32_t *dst = staged ? reinterpret_cast<int32_t *>(s_list) : out;
    for (int w0 = wbeg; w0 < min(nwords, wbeg + per_warp); w0 += 32) {   // uniform per warp
        const int wd = w0 + lane;
        unsigned bits = wd < nwords ? bitmap[wd] : 0u;
        const unsigned c = __popc(bits);
        unsigned incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        unsigned posn = run + incl - c;
        run += __shfl_sync(0xffffffffu, incl, 31);
        while (bits) {
            const int bpos = __ffs(bits) - 1;
            bits &= bits - 1;
            if (posn < (unsigned)p.k) dst[posn] = wd * 32 + bpos;
            ++posn;
        }
    }
    if (staged) {
        __syncthreads();
        for (int t = tid; t < p.k; t += THREADS) out[t] = t < k_row ? dst[t] : -1;
    } else {
        for (int t = k_row + tid; t < p.k; t += THREADS) out[t] = -1;
    }
    // a list with a repeated key (never written by the sweep) would select fewer keys than wanted: leave such a row to the redo
    if (total_sel != (unsigned)k_row && tid == 0) flag[blockIdx.x] = 1;
}

}  // namespace

cudaError_t launch_filter_thresholds(const Params &p, const float *sample, int64_t stride, int64_t row0, int64_t n_rows,
                                     int samp, int cap, uint32_t *tau_key, int *flag, cudaStream_t st)
{
    if (n_rows == 0) return cudaSuccess;
    const unsigned n = (unsigned)n_rows;
    // sample sizes that occur among the rows of this block (known on the host when the positions are)
    int ns_min = 0, ns_max = filter_sample_width(p, samp);
    if (!p.q_start && !p.kv_lens && row0 / p.Lq == (row0 + n_rows - 1) / p.Lq) {
        auto nk = [&](int64_t i) { const int64_t v = (int64_t)p.Lk - p.Lq + i - p.w + 1; return (int)(v < 0 ? 0 : (v > p.Lk ? p.Lk : v)); };
        ns_min = sample_size(nk(row0 % p.Lq), samp);
        ns_max = sample_size(nk((row0 + n_rows - 1) % p.Lq), samp);
    }
    // class by the size of the row's sample (every row is taken by exactly one launch); a sample gets no more warps
    // than it fills.  Classes that no row of the block falls into are not launched.
    auto go = [&](auto kern, int threads, int e, int lo, int hi) -> cudaError_t {
        if (ns_max <= lo || ns_min > hi) return cudaSuccess;
        const size_t smem = (size_t)threads * e * sizeof(uint32_t);
        if (smem > 24 * 1024) {   // static shared memory counts against the 48 KB default too
            const cudaError_t e2 = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e2 != cudaSuccess) return e2;
        }
        kern<<<n, threads, smem, st>>>(p, sample, stride, row0, lo, hi, samp, cap, tau_key, flag);
        count_launch();
        return cudaSuccess;
    };
    cudaError_t e = go(k_sample_tau<64, 16>, 64, 16, -1, 1024);
    if (e == cudaSuccess) e = go(k_sample_tau<128, 16>, 128, 16, 1024, 2048);
    if (e == cudaSuccess) e = go(k_sample_tau<256, 16>, 256, 16, 2048, 4096);
    if (e == cudaSuccess) e = go(k_sample_tau<256, 32>, 256, 32, 4096, 8192);
    if (e == cudaSuccess) e = go(k_sample_tau<512, 32>, 512, 32, 8192, 16384);
    if (e == cudaSuccess) e = go(k_sample_tau<512, 64>, 512, 64, 16384, 32768);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

// final selection from the candidate lists; rows whose lists are unusable get flag[row] = 1
cudaError_t launch_filter_select(const Params &p, const void *cand, const int *count, int cap,
                                 int32_t *idx, int64_t row0, int64_t n_rows, int *flag, cudaStream_t st)
{
    if (n_rows == 0) return cudaSuccess;
    const unsigned n = (unsigned)n_rows;
    const size_t bm = cached_bitmap_bytes(p.Lk);   // one bit per key of the row, then the list (later the staged output row)
    auto go = [&](auto kern, int threads, int e) -> cudaError_t {
        const size_t smem = bm + (size_t)kCandList * sizeof(uint32_t) + (size_t)threads * e * sizeof(int32_t);
        if (smem > 24 * 1024) {   // static shared memory counts against the 48 KB default too
            const cudaError_t e2 = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e2 != cudaSuccess) return e2;
        }
        kern<<<n, threads, smem, st>>>(p, static_cast<const int2 *>(cand), count, cap, idx, row0, flag);
        count_launch();
        return cudaSuccess;
    };
    // a thread group of THREADS / 4 takes one sub-list of cap / 4 slots, E slots per thread
    cudaError_t e;
    if (cap <= 2048) e = go(k_cand_select<128, 16>, 128, 16);
    else if (cap <= 4096) e = go(k_cand_select<256, 16>, 256, 16);
    else if (cap <= 8192) e = go(k_cand_select<256, 32>, 256, 32);
    else e = go(k_cand_select<512, 64>, 512, 64);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

cudaError_t launch_select_recompute(const Params &p, const void *Q, const void *K, const float *LSE, int32_t *idx,
                                    int64_t row0, int64_t n_rows, const int *flag, cudaStream_t st)
{
    if (n_rows == 0) return cudaSuccess;
    const size_t smem = sizeof(float) * ((size_t)p.G * 128 + p.G);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)std::min<int64_t>((n_rows + kRedoChunk - 1) / kRedoChunk, (int64_t)8 * sms);
    k_select_recompute<<<grid, 256, smem, st>>>(p, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)K, LSE, idx, row0, n_rows,
                                                flag);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hs2
