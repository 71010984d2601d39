// Token-level top-k outside the forced window on a materialised score row (Section 3.3).
//
// One CTA per (batch, KV head, query) row.  The row's candidates are keys 0 .. pos-w.  An exact
// radix select on order-preserving 32-bit keys (four 8-bit digits, most significant first) finds
// the value of the take-th largest score and how many candidates equal to it are still needed;
// one ordered compaction pass then writes the kept indices in ascending key order, taking equal
// scores from the lowest index upwards.  The result depends only on the score bits.
#include <cooperative_groups.h>

#include "hs2_common.cuh"

namespace hs2 {
namespace {

constexpr int kItems = 4;                    // consecutive scores per thread per step
constexpr unsigned kListCap = 2048;          // threshold-bin candidates kept in shared memory (cached variant)

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

// ---- rows that fit in registers: THREADS x E candidates, read once ------------------------------
// Thread t owns the E consecutive candidates E t .. E t + E - 1, so the ascending-index order of the
// output is (thread, element) order and the ordered compaction needs a single block scan.  The radix
// digits are taken below the common leading bits of the row's smallest and largest key, which makes
// the first round spread the candidates over all 256 bins (log-probabilities share their top bits).
template <int THREADS, int E, bool VEC>
__global__ void __launch_bounds__(THREADS, THREADS <= 256 ? 3 : 1)
k_topk_cached(const Params p, const float *__restrict__ scores, int64_t score_stride, int32_t *__restrict__ idx,
              int64_t row0, int nc_lo, int nc_hi)
{
    constexpr int WARPS = THREADS / 32;
    __shared__ unsigned hist[256];
    __shared__ unsigned s_warp[WARPS];
    __shared__ unsigned s_min[WARPS], s_max[WARPS];
    __shared__ unsigned s_prefix, s_need, s_cnt;
    __shared__ uint32_t s_list[kListCap];

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
    const int j0 = tid * E;
    uint32_t key[E];
    unsigned kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
    for (int e4 = 0; e4 < E; e4 += 4) {
        if (VEC && j0 + e4 + 4 <= nc) {
            const float4 v = __ldg(reinterpret_cast<const float4 *>(srow + j0 + e4));
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
#pragma unroll
    for (int w = 0; w < WARPS; ++w) { kmin = min(kmin, s_min[w]); kmax = max(kmax, s_max[w]); }

    // bits above `hi` are equal in every candidate; resolve the rest 8 bits at a time
    int hi = 32 - __clz(kmin ^ kmax);          // 0 when all candidates are equal
    unsigned prefix = hi >= 32 ? 0u : (kmax >> hi);
    unsigned need = (unsigned)take;
    bool on_list = false;                      // later rounds run on the threshold bin's candidates only
    unsigned n_list = 0;
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
        } else {
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const bool live = (j0 + e < nc) && (hi >= 32 || (key[e] >> hi) == prefix);
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
        const bool collect = !on_list && hi > 0 && in_bin <= kListCap;
        __syncthreads();   // every thread has read hist[digit] before the next round zeroes the histogram
        if (collect) {
            // every candidate that can still be the take-th largest sits in this bin (at most kListCap of them)
#pragma unroll
            for (int e = 0; e < E; ++e)
                if (j0 + e < nc && (key[e] >> hi) == prefix) {
                    const unsigned slot = atomicAdd(&s_cnt, 1u);
                    if (slot < kListCap) s_list[slot] = key[e];
                }
            __syncthreads();
            on_list = true;
            n_list = min(s_cnt, kListCap);
        }
    }
    const uint32_t tau = hi == 0 && kmin == kmax ? kmax : prefix;   // key of the take-th largest candidate
    const unsigned need_eq = need;                                   // equal keys kept, lowest indices first

    // ---- ordered compaction with one block scan
    unsigned n_gt = 0, n_eq = 0;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        const bool ok = j0 + e < nc;
        n_gt += ok && key[e] > tau;
        n_eq += ok && key[e] == tau;
    }
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
    for (int t = take + tid; t < p.k; t += THREADS) out[t] = -1;
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
#pragma unroll
    for (int e4 = 0; e4 < E; e4 += 4) {
        if (VEC && j0 + e4 + 4 <= nc) {
            const float4 v = __ldg(reinterpret_cast<const float4 *>(srow + j0 + e4));
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
constexpr TopkClass kClasses[6] = {{-1, 8192}, {8192, 32768}, {32768, 65536}, {65536, 131072}, {131072, 262144},
                                   {262144, 0x7fffffff}};

template <bool VEC>
void launch_class(int c, const Params &p, const float *scores, int64_t score_stride, int32_t *idx, int64_t row0,
                  int64_t n_rows, cudaStream_t st)
{
    const int lo = kClasses[c].lo, hi = kClasses[c].hi;
    const unsigned n = (unsigned)n_rows;
#ifdef HS2_TOPK_NO_CLUSTER
    if (c >= 2 && c <= 4) c = 5;   // tuning builds: long rows on the streaming kernel
#endif
    switch (c) {
        case 0: k_topk_cached<256, 32, VEC><<<n, 256, 0, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
        case 1: k_topk_cached<512, 64, VEC><<<n, 512, 0, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
        case 2: k_topk_cluster<2, VEC><<<n * 2, 512, 0, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
        case 3: k_topk_cluster<4, VEC><<<n * 4, 512, 0, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
        case 4: k_topk_cluster<8, VEC><<<n * 8, 512, 0, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
        default: k_topk<1024, kItems, false, VEC><<<n, 1024, 0, st>>>(p, scores, score_stride, idx, row0, lo, hi); break;
    }
    count_launch();
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
    for (int c = 0; c < 6; ++c) {
        if (nc_max <= kClasses[c].lo || nc_min > kClasses[c].hi) continue;   // no row of the block falls in this class
        if (vec) launch_class<true>(c, p, scores, score_stride, idx, row0, n_rows, st);
        else launch_class<false>(c, p, scores, score_stride, idx, row0, n_rows, st);
    }
    return cudaGetLastError();
}

}  // namespace hs2
