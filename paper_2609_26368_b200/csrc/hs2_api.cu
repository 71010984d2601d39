// C ABI of the hs2 library: argument validation, default resolution, workspace carving, dispatch.
#include <math.h>

#include <atomic>

#include "hs2_common.cuh"

namespace hs2 {

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

namespace {

thread_local int g_last_cuda_error = 0;

hs2_status cuda_fail(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    return HS2_ERR_CUDA;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

#ifndef HS2_STRIP_CAP_MB
#define HS2_STRIP_CAP_MB 1024
#endif
constexpr size_t kStripCapBytes = (size_t)HS2_STRIP_CAP_MB << 20;   // bound on the score strips of one launch

// Validate the host-visible part of a problem and resolve defaults.
hs2_status resolve(const hs2_problem *hp, bool need_tensors, Params *out)
{
    if (!hp) return HS2_ERR_INVALID_ARG;
    if (hp->batch <= 0 || hp->n_kv_heads <= 0 || hp->q_len <= 0 || hp->kv_len <= 0) return HS2_ERR_INVALID_ARG;
    if (hp->k_sel < 0 || hp->window < 0) return HS2_ERR_INVALID_ARG;
    if (hp->k_sel == 0 && hp->window == 0) return HS2_ERR_INVALID_ARG;   // every attended set would be empty
    Params p{};
    p.B = hp->batch; p.Hkv = hp->n_kv_heads; p.Lq = hp->q_len; p.Lk = hp->kv_len;
    p.k = hp->k_sel; p.w = hp->window;
    p.q_start = hp->q_start; p.kv_lens = hp->kv_lens;
    p.blk = hp->select_block > 1 ? hp->select_block : 1;
    if (hp->select_block < 0 || (p.blk > 1 && (hp->k_sel % p.blk != 0 || p.blk > 1024))) return HS2_ERR_INVALID_ARG;
    p.Hq = hp->n_q_heads; p.D = hp->head_dim;
    if (need_tensors) {
        if (hp->n_q_heads <= 0 || hp->n_q_heads % hp->n_kv_heads != 0 || hp->head_dim <= 0) return HS2_ERR_INVALID_ARG;
        if (hp->dtype != HS2_F32 && hp->dtype != HS2_BF16) return HS2_ERR_INVALID_ARG;
        if (!(hp->softmax_scale >= 0.f) || isinf(hp->softmax_scale)) return HS2_ERR_INVALID_ARG;
        if (hp->head_dim > 256) return HS2_ERR_UNSUPPORTED;
        p.G = p.Hq / p.Hkv;
        p.scale = hp->softmax_scale > 0.f ? hp->softmax_scale : 1.0f / sqrtf((float)p.D);
        p.scale_log2 = p.scale * kLog2e;
        auto strides = [](const int64_t s[3], int64_t L, int64_t H, int64_t D, int64_t &sb, int64_t &st, int64_t &sh) {
            if (s[0] == 0 && s[1] == 0 && s[2] == 0) { sh = D; st = H * D; sb = L * H * D; return true; }
            sb = s[0]; st = s[1]; sh = s[2];
            return s[2] >= D && s[1] >= 0 && s[0] >= 0;
        };
        if (!strides(hp->q_stride, p.Lq, p.Hq, p.D, p.qs_b, p.qs_t, p.qs_h)) return HS2_ERR_INVALID_ARG;
        if (!strides(hp->kv_stride, p.Lk, p.Hkv, p.D, p.ks_b, p.ks_t, p.ks_h)) return HS2_ERR_INVALID_ARG;
        if (!strides(hp->o_stride, p.Lq, p.Hq, p.D, p.os_b, p.os_t, p.os_h)) return HS2_ERR_INVALID_ARG;
        {   // scales of an FP8 cache: one float per (batch, token, KV head)
            const int64_t *s = hp->kv_scale_stride;
            if (s[0] == 0 && s[1] == 0 && s[2] == 0) { p.ss_h = 1; p.ss_t = p.Hkv; p.ss_b = (int64_t)p.Lk * p.Hkv; }
            else if (s[0] >= 0 && s[1] >= 0 && s[2] >= 1) { p.ss_b = s[0]; p.ss_t = s[1]; p.ss_h = s[2]; }
            else return HS2_ERR_INVALID_ARG;
        }
    } else {
        p.G = 1;
    }
    *out = p;
    return HS2_OK;
}

int64_t select_rows(const Params &p) { return (int64_t)p.B * p.Hkv * p.Lq; }

// token-level top-k (Section 3.3) or the block-level variant of the paper's first ablation
cudaError_t launch_select(const Params &p, const float *scores, int64_t stride, int32_t *idx, int64_t r0, int64_t n,
                          cudaStream_t st)
{
    return p.blk > 1 ? launch_block_select(p, scores, stride, idx, r0, n, st) : launch_topk(p, scores, stride, idx, r0, n, st);
}

size_t strip_row_bytes(const Params &p) { return align_up((size_t)p.Lk * sizeof(float), 16); }

size_t full_select_ws_bytes(const Params &p)
{
    const size_t row = strip_row_bytes(p);
    size_t rows = (size_t)select_rows(p);
    const size_t cap_rows = kStripCapBytes / row > 0 ? kStripCapBytes / row : 1;
    if (rows > cap_rows) rows = cap_rows;
    return align_up(rows * row, 256);
}

// Decode-shaped full layer (one query per sequence) on the mma.sync gather kernel: the sweep over the cache keeps the
// raw q.k products, so that the selection scores need no second pass over K.  Scratch: [sweep's own scratch][raw
// products: B * Hq * Lk floats][score rows: B * Hkv rows].
struct DecodeFusedPlan { size_t off_raw, off_strip, total; bool ok; };
constexpr size_t kRawCapBytes = (size_t)2 << 30;   // beyond this the layer sweeps K twice instead
DecodeFusedPlan decode_fused_plan(const Params &pd, size_t sweep_ws)
{
    DecodeFusedPlan f;
    f.ok = (size_t)pd.B * pd.Hq * pd.Lk * sizeof(float) <= kRawCapBytes;
    f.off_raw = align_up(sweep_ws, 256);
    f.off_strip = f.off_raw + align_up((size_t)pd.B * pd.Hq * pd.Lk * sizeof(float), 256);
    f.total = f.off_strip + align_up((size_t)pd.B * pd.Hkv * strip_row_bytes(pd), 256);
    return f;
}

// ---- filtered selection (sampled threshold -> ordered candidate lists -> select) ----
constexpr int kFilterSamp = 16;             // every 16th key tile is scored for the threshold (every 8th: 6 ms more at 128K)
// The filtered path wins when rows are long (measured, full layer with selection, filtered vs strips: 2 x 32768 keys
// 30.8 vs 38.0 ms, 2 x 20480 keys 13.4 vs 14.6 ms, 2 x 16384 keys 9.1 vs 8.7 ms, 8192 keys 1.32 vs 1.10 ms): shorter
// contexts keep the strips.
std::atomic<int> g_filter_min_keys{18432};
std::atomic<int> g_disable_tc5{0};          // testing knob: run the mma.sync kernels instead of the tcgen05 ones
constexpr size_t kFilterBigCap = (size_t)1 << 30;

struct FilterPlan {
    bool ok;
    int cap;          // candidates kept per row
    int ns_w;         // sampled scores per row (padded to whole tiles)
    size_t per_row;   // bytes of the big region per row (sample strip, later the candidate lists)
};

FilterPlan filter_plan(const Params &p, hs2_dtype dt)
{
    FilterPlan f{};
    // expected list length: samp * r with r the threshold rank at the thinnest sampling (1/samp), standard deviation
    // samp * sqrt(r).  The list is kept as four sub-lists (one per quarter of a key tile), each a quarter of the
    // list give or take the binomial split: capacity = mean + 6 standard deviations per sub-list.
    const double m = (double)p.k / kFilterSamp, r = m + 5.0 * sqrt(m) + 2.0;
    const double mean = kFilterSamp * r, sd_sub = sqrt(kFilterSamp * kFilterSamp * r / 16.0 + 3.0 * mean / 16.0);
    const int want = (int)(mean + 4.0 * 6.0 * sd_sub) + 64;
    f.cap = ((want > 1024 ? want : 1024) + 255) / 256 * 256;
    f.ns_w = filter_sample_width(p, kFilterSamp);
    f.per_row = align_up((size_t)f.ns_w * 4, 16);
    if ((size_t)f.cap * 8 > f.per_row) f.per_row = (size_t)f.cap * 8;
    f.ok = p.k > 0 && p.blk == 1 && !g_disable_tc5.load(std::memory_order_relaxed) && scores_filter_supported(p, dt) && f.cap <= 32768 && f.ns_w <= 32768 && p.Lk > f.cap &&
           p.Lk >= g_filter_min_keys.load(std::memory_order_relaxed) && select_rows(p) >= 1024;
    return f;
}

int64_t filter_block_rows(const FilterPlan &f, int64_t rows, size_t ws_bytes)
{
    const size_t budget = ws_bytes < kFilterBigCap + (size_t)(16 << 20) ? ws_bytes : kFilterBigCap + (size_t)(16 << 20);
    if (budget < 4096) return 0;
    int64_t r = (int64_t)((budget - 4096) / (f.per_row + 24));
    return r > rows ? rows : r;
}

size_t filter_ws_bytes(const FilterPlan &f, int64_t rows)
{
    int64_t r = (int64_t)(kFilterBigCap / f.per_row);
    if (r > rows) r = rows;
    if (r < 1) r = 1;
    return align_up((size_t)r * (f.per_row + 24) + 4096, 256);
}

bool ws_ok(const void *ws, size_t ws_bytes, size_t need)
{
    if (need == 0) return true;
    return ws != nullptr && ws_bytes >= need && reinterpret_cast<uintptr_t>(ws) % 256 == 0;
}

bool aligned16(const void *a, const void *b, const void *c, const void *d)
{
    return ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) | reinterpret_cast<uintptr_t>(c) |
             reinterpret_cast<uintptr_t>(d)) & 15) == 0;
}

hs2_status check_device()
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    return HS2_OK;
}

// the score sweep: tcgen05 where it applies, else mma.sync, else the generic kernel
cudaError_t launch_scores(const Params &p, hs2_dtype dt, bool mma, bool aligned, const void *Q, const void *K, const float *LSE,
                          float *out, int64_t out_stride, int64_t row0, int64_t n_rows, bool all_visible, cudaStream_t st)
{
    cudaError_t e = cudaErrorNotSupported;
#ifndef HS2_NO_TC5
    if (aligned && !g_disable_tc5.load(std::memory_order_relaxed) && scores_tc5_supported(p, dt)) e = launch_scores_tc5(p, Q, K, LSE, out, out_stride, row0, n_rows, all_visible, st);
#endif
    if (e == cudaErrorNotSupported)
        e = mma ? launch_scores_mma(p, Q, K, LSE, out, out_stride, row0, n_rows, all_visible, st)
                : launch_scores_generic(p, dt, Q, K, LSE, out, out_stride, row0, n_rows, all_visible, st);
    return e;
}

// the gate is read with the 16-byte accesses of the output it scales
bool gate_aligned(const void *gate) { return (reinterpret_cast<uintptr_t>(gate) & 15u) == 0; }

// The mma.sync gather kernel covers groups of up to 8 heads.  A bf16 head_dim-128 group of 16 runs on it as two
// sub-groups of 8 that read the same KV head (the rows come from L2 the second time); measured 2x faster than the
// tcgen05 gather kernel at this small head_dim.  Larger groups stay on the tcgen05 kernel.
void split_into_subgroups(Params *p, hs2_dtype dt)
{
    if (dt == HS2_BF16 && p->D == 128 && p->G == 16) {
        p->share = 2;
        p->Hkv *= 2;
        p->G = 8;
    }
}

hs2_status sparse_common(const hs2_problem *hp, const void *Q, const void *K, const void *V, const int32_t *idx,
                         void *O, Params *p)
{
    hs2_status s = resolve(hp, true, p);
    if (s != HS2_OK) return s;
    if (!Q || !K || !V || !O) return HS2_ERR_INVALID_ARG;
    if (p->k > 0 && !idx) return HS2_ERR_INVALID_ARG;
    return HS2_OK;
}

}  // namespace
}  // namespace hs2

using namespace hs2;

extern "C" {

size_t hs2_workspace_bytes(const hs2_problem *hp, hs2_op op)
{
    Params p;
    switch (op) {
        case HS2_OP_FULL_ATTN_SELECT:
            if (resolve(hp, true, &p) != HS2_OK) return 0;
            {
                size_t need = p.k > 0 ? full_select_ws_bytes(p) : 0;
                const FilterPlan fp = filter_plan(p, hp->dtype);
                if (fp.ok) {
                    const size_t fneed = filter_ws_bytes(fp, select_rows(p));
                    if (fneed > need) need = fneed;
                }
                if (p.Lq == 1) {   // the decode-shaped layer may split over the keys
                    Params pd = p;
                    pd.k = 0; pd.w = p.Lk;
                    const DecodeFusedPlan fu = decode_fused_plan(pd, sparse_mma_supported(p, hp->dtype) ? sparse_mma_decode_ws_bytes(pd) : 0);
                    const size_t dec = sparse_mma_supported(p, hp->dtype)         ? (fu.ok ? fu.total : sparse_mma_decode_ws_bytes(pd))
                                       : sparse_tc5_supported_shape(pd, hp->dtype) ? sparse_tc5_ws_bytes(pd)
                                                                                   : 0;
                    if (dec > need) need = dec;
                }
                return need;
            }
        case HS2_OP_TOPK_SELECT:
        case HS2_OP_SPARSE_ATTN_PREFILL:
            return 0;
        case HS2_OP_FULL_ATTN_SELECT_FP8KV:
            if (resolve(hp, true, &p) != HS2_OK) return 0;
            if (p.Lq != 1 || p.k == 0) return 0;
            {
                Params pd = p;
                pd.k = 0; pd.w = p.Lk;
                if (!sparse_fp8_supported(pd, hp->dtype))   // large groups / head_dim 256: one score row per (sequence, KV head)
                    return sparse_tc5_fp8_supported(pd, hp->dtype) ? align_up((size_t)p.B * p.Hkv * strip_row_bytes(p), 256) : 0;
                const DecodeFusedPlan fu = decode_fused_plan(pd, 0);
                return fu.ok ? fu.total : 0;
            }
        case HS2_OP_SPARSE_ATTN_DECODE:
            if (resolve(hp, true, &p) != HS2_OK) return 0;
            if (p.Lq != 1) return 0;
            split_into_subgroups(&p, hp->dtype);
            if (sparse_mma_supported(p, hp->dtype)) return sparse_mma_decode_ws_bytes(p);
            return sparse_tc5_supported_shape(p, hp->dtype) ? sparse_tc5_ws_bytes(p) : 0;
    }
    return 0;
}

hs2_status hs2_full_attn_select(const hs2_problem *hp, const void *Q, const void *K, const void *V, void *O,
                                float *LSE, int32_t *idx, float *scores_dbg, void *ws, size_t ws_bytes,
                                void *cuda_stream)
{
    Params p;
    hs2_status s = resolve(hp, true, &p);
    if (s != HS2_OK) return s;
    if (!Q || !K || !V || !O || !LSE) return HS2_ERR_INVALID_ARG;
    const bool want_sel = idx != nullptr && p.k > 0;
    const size_t row_bytes = strip_row_bytes(p);
    // any aligned buffer holding at least one strip row works; a smaller buffer only means more launches
    if (want_sel && !scores_dbg && !ws_ok(ws, ws_bytes, row_bytes)) return HS2_ERR_WORKSPACE_TOO_SMALL;
    if ((s = check_device()) != HS2_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const hs2_dtype dt = hp->dtype;
    const bool mma = full_mma_supported(p, dt) && aligned16(Q, K, V, O);
    cudaError_t e;
    // One query per sequence: the layer is a memory-bound sweep over the whole cache.  That is the
    // sparse decode kernel with an empty index list and a window that covers the context.
    bool as_decode = p.Lq == 1 && sparse_mma_supported(p, dt) && aligned16(Q, K, V, O);
    Params pd = p;
    pd.k = 0; pd.w = p.Lk;
    if (as_decode && !ws_ok(ws, ws_bytes, sparse_mma_decode_ws_bytes(pd))) as_decode = false;
    if (as_decode) {
        const bool want_sel_now = idx != nullptr && p.k > 0 && !scores_dbg;
        const DecodeFusedPlan fu = decode_fused_plan(pd, sparse_mma_decode_ws_bytes(pd));
        if (want_sel_now && fu.ok && ws_bytes >= fu.total && (int64_t)p.B * p.Hkv <= 65535) {
            float *raw = reinterpret_cast<float *>(static_cast<char *>(ws) + fu.off_raw);
            float *strip = reinterpret_cast<float *>(static_cast<char *>(ws) + fu.off_strip);
            e = launch_sparse_mma_decode(pd, Q, K, V, nullptr, nullptr, O, LSE, ws, ws_bytes, st, raw);
            if (e == cudaSuccess) {
                const int64_t stride = (int64_t)(strip_row_bytes(p) / sizeof(float));
                if ((e = launch_scores_from_raw(p, raw, LSE, strip, stride, st)) != cudaSuccess) return cuda_fail(e);
                if ((e = launch_select(p, strip, stride, idx, 0, select_rows(p), st)) != cudaSuccess) return cuda_fail(e);
                return HS2_OK;
            }
            if (e != cudaErrorNotSupported) return cuda_fail(e);
            (void)cudaGetLastError();
        }
        e = launch_sparse_mma_decode(pd, Q, K, V, nullptr, nullptr, O, LSE, ws, ws_bytes, st);
    } else {
        e = cudaErrorNotSupported;
        // the same idea for large head groups: the tcgen05 gather kernel, keys split over CTAs through the scratch
        if (p.Lq == 1 && !g_disable_tc5.load(std::memory_order_relaxed) && sparse_tc5_supported(pd, dt) && aligned16(Q, K, V, O)) {
            const bool ws_usable = ws != nullptr && (reinterpret_cast<uintptr_t>(ws) & 15u) == 0;
            e = launch_sparse_tc5(pd, Q, K, V, nullptr, nullptr, O, LSE, ws_usable ? ws : nullptr, ws_usable ? ws_bytes : 0, st);
        }
#ifndef HS2_NO_TC5
        if (e == cudaErrorNotSupported && !g_disable_tc5.load(std::memory_order_relaxed) && full_attn_tc5_supported(p, dt) &&
            aligned16(Q, K, V, O))
            e = launch_full_attn_tc5(p, Q, K, V, O, LSE, st);
#endif
        if (e == cudaErrorNotSupported)
            e = mma ? launch_full_attn_mma(p, Q, K, V, O, LSE, st) : launch_full_attn_generic(p, dt, Q, K, V, O, LSE, st);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    if (!want_sel && !scores_dbg) return HS2_OK;

    const int64_t rows = select_rows(p);
    constexpr int64_t kMaxBlockRows = 262144;   // keeps the score kernels' grid.y inside its limit
    if (scores_dbg) {
        // scores for every visible key go straight to the caller's tensor; the selection reads them from there
        for (int64_t r0 = 0; r0 < rows; r0 += kMaxBlockRows) {
            const int64_t n = rows - r0 < kMaxBlockRows ? rows - r0 : kMaxBlockRows;
            float *dst = scores_dbg + r0 * p.Lk;
            e = launch_scores(p, dt, mma, aligned16(Q, K, V, O), Q, K, LSE, dst, p.Lk, r0, n, true, st);
            if (e != cudaSuccess) return cuda_fail(e);
            if (want_sel && (e = launch_select(p, dst, p.Lk, idx, r0, n, st)) != cudaSuccess) return cuda_fail(e);
        }
        return HS2_OK;
    }
    // Filtered path: a 1/8-sampled sweep gives every row a threshold that (with verification) lies below its
    // k-th score; the main sweep then keeps only the (score, key) pairs at or above it, in key order, and the
    // selection runs on those short lists.  Rows whose list came out too short or too long are redone exactly.
    const FilterPlan fp = filter_plan(p, dt);
    const bool al = aligned16(Q, K, V, O);
    if (fp.ok && al && reinterpret_cast<uintptr_t>(ws) % 256 == 0) {
        int64_t block = filter_block_rows(fp, rows, ws_bytes);
        if (block > kMaxBlockRows) block = kMaxBlockRows;
        if (block >= (rows < 1024 ? rows : 1024)) {
            char *base = (char *)ws;
            uint32_t *tau = (uint32_t *)base;
            int *flag = (int *)(base + (size_t)block * 4);
            int *count = (int *)(base + (size_t)block * 8);   // four sub-list counts per row
            char *big = base + align_up((size_t)block * 24, 256);
            float *sample = (float *)big;
            void *cand = big;   // block * cap records of (score, key), 8 bytes each
            bool usable = true;
            for (int64_t r0 = 0; r0 < rows && usable; r0 += block) {
                const int64_t n = rows - r0 < block ? rows - r0 : block;
                e = launch_scores_sampled_tc5(p, Q, K, LSE, sample, fp.ns_w, r0, n, kFilterSamp, st);
                if (e == cudaErrorNotSupported && r0 == 0) { usable = false; break; }   // nothing launched yet: use the strips
                if (e != cudaSuccess) return cuda_fail(e);
                if ((e = launch_filter_thresholds(p, sample, fp.ns_w, r0, n, kFilterSamp, fp.cap, tau, flag, st)) != cudaSuccess) return cuda_fail(e);
                if ((e = launch_scores_filter_tc5(p, Q, K, LSE, r0, n, tau, cand, count, fp.cap, st)) != cudaSuccess) return cuda_fail(e);
                if ((e = launch_filter_select(p, cand, count, fp.cap, idx, r0, n, flag, st)) != cudaSuccess) return cuda_fail(e);
                if ((e = launch_select_recompute(p, Q, K, LSE, idx, r0, n, flag, st)) != cudaSuccess) return cuda_fail(e);
            }
            if (usable) return HS2_OK;
        }
    }
    // bounded strips: score a block of query rows into the workspace, select from it, move on
    const int64_t stride = (int64_t)(row_bytes / sizeof(float));
    int64_t block = (int64_t)((ws_bytes < kStripCapBytes ? ws_bytes : kStripCapBytes) / row_bytes);
    if (block < 1) block = 1;
    if (block > kMaxBlockRows) block = kMaxBlockRows;
    if (block > rows) block = rows;
    float *strip = (float *)ws;
    for (int64_t r0 = 0; r0 < rows; r0 += block) {
        const int64_t n = rows - r0 < block ? rows - r0 : block;
        e = launch_scores(p, dt, mma, al, Q, K, LSE, strip, stride, r0, n, false, st);
        if (e != cudaSuccess) return cuda_fail(e);
        if ((e = launch_select(p, strip, stride, idx, r0, n, st)) != cudaSuccess) return cuda_fail(e);
    }
    return HS2_OK;
}

hs2_status hs2_topk_select(const hs2_problem *hp, const float *scores, int32_t *idx, void *ws, size_t ws_bytes,
                           void *cuda_stream)
{
    (void)ws; (void)ws_bytes;
    Params p;
    hs2_status s = resolve(hp, false, &p);
    if (s != HS2_OK) return s;
    if (p.k > 0 && (!scores || !idx)) return HS2_ERR_INVALID_ARG;
    if ((s = check_device()) != HS2_OK) return s;
    cudaError_t e = launch_select(p, scores, p.Lk, idx, 0, select_rows(p), (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? HS2_OK : cuda_fail(e);
}

static hs2_status sparse_prefill_impl(const hs2_problem *hp, const void *Q, const void *K, const void *V, const int32_t *idx,
                                      const float *sink, const void *gate, void *O, float *LSE, void *ws, size_t ws_bytes,
                                      void *cuda_stream)
{
    (void)ws; (void)ws_bytes;
    Params p;
    hs2_status s = sparse_common(hp, Q, K, V, idx, O, &p);
    if (s != HS2_OK) return s;
    p.gate = gate;
    if ((s = check_device()) != HS2_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaErrorNotSupported;
    Params pm = p;   // the mma.sync kernel's view: a group of 16 as two sub-groups of 8
    split_into_subgroups(&pm, hp->dtype);
    if (sparse_mma_supported(pm, hp->dtype) && aligned16(Q, K, V, O) && gate_aligned(gate)) {
        e = launch_sparse_mma_prefill(pm, Q, K, V, idx, sink, O, LSE, st);
    } else {
        // large head groups (the paper's 64 heads per KV head): the gather tile is a dense contraction
        if (!g_disable_tc5.load(std::memory_order_relaxed) && sparse_tc5_supported(p, hp->dtype) && aligned16(Q, K, V, O) && gate_aligned(gate))
            e = launch_sparse_tc5(p, Q, K, V, idx, sink, O, LSE, nullptr, 0, st);
        if (e == cudaErrorNotSupported) {
            (void)cudaGetLastError();
            e = launch_sparse_generic(p, hp->dtype, Q, K, V, idx, sink, O, LSE, st);
        }
    }
    return e == cudaSuccess ? HS2_OK : cuda_fail(e);
}

hs2_status hs2_sparse_attn_prefill(const hs2_problem *hp, const void *Q, const void *K, const void *V,
                                   const int32_t *idx, const float *sink, void *O, float *LSE, void *ws,
                                   size_t ws_bytes, void *cuda_stream)
{
    return sparse_prefill_impl(hp, Q, K, V, idx, sink, nullptr, O, LSE, ws, ws_bytes, cuda_stream);
}

hs2_status hs2_sparse_attn_prefill_gated(const hs2_problem *hp, const void *Q, const void *K, const void *V,
                                         const int32_t *idx, const float *sink, const void *gate, void *O, float *LSE,
                                         void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!gate) return HS2_ERR_INVALID_ARG;
    return sparse_prefill_impl(hp, Q, K, V, idx, sink, gate, O, LSE, ws, ws_bytes, cuda_stream);
}

static hs2_status sparse_decode_impl(const hs2_problem *hp, const void *Q, const void *K, const void *V, const int32_t *idx,
                                     const float *sink, const void *gate, void *O, float *LSE, void *ws, size_t ws_bytes,
                                     void *cuda_stream)
{
    Params p;
    hs2_status s = sparse_common(hp, Q, K, V, idx, O, &p);
    if (s != HS2_OK) return s;
    p.gate = gate;
    if (p.Lq != 1) return HS2_ERR_INVALID_ARG;
    Params pm = p;
    split_into_subgroups(&pm, hp->dtype);
    const bool mma = sparse_mma_supported(pm, hp->dtype) && aligned16(Q, K, V, O) && gate_aligned(gate);
    if (mma && !ws_ok(ws, ws_bytes, sparse_mma_decode_ws_bytes(pm))) return HS2_ERR_WORKSPACE_TOO_SMALL;
    if ((s = check_device()) != HS2_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaErrorNotSupported;
    if (mma) {
        e = launch_sparse_mma_decode(pm, Q, K, V, idx, sink, O, LSE, ws, ws_bytes, st);
    } else {
        // large head groups: the tcgen05 gather kernel, its keys split over CTAs when the scratch allows
        if (!g_disable_tc5.load(std::memory_order_relaxed) && sparse_tc5_supported(p, hp->dtype) && aligned16(Q, K, V, O) && gate_aligned(gate)) {
            const bool ws_usable = ws != nullptr && (reinterpret_cast<uintptr_t>(ws) & 15u) == 0;
            e = launch_sparse_tc5(p, Q, K, V, idx, sink, O, LSE, ws_usable ? ws : nullptr, ws_usable ? ws_bytes : 0, st);
        }
        if (e == cudaErrorNotSupported) {
            (void)cudaGetLastError();
            e = launch_sparse_generic(p, hp->dtype, Q, K, V, idx, sink, O, LSE, st);
        }
    }
    return e == cudaSuccess ? HS2_OK : cuda_fail(e);
}

hs2_status hs2_sparse_attn_decode(const hs2_problem *hp, const void *Q, const void *K, const void *V,
                                  const int32_t *idx, const float *sink, void *O, float *LSE, void *ws,
                                  size_t ws_bytes, void *cuda_stream)
{
    return sparse_decode_impl(hp, Q, K, V, idx, sink, nullptr, O, LSE, ws, ws_bytes, cuda_stream);
}

hs2_status hs2_sparse_attn_decode_gated(const hs2_problem *hp, const void *Q, const void *K, const void *V,
                                        const int32_t *idx, const float *sink, const void *gate, void *O, float *LSE,
                                        void *ws, size_t ws_bytes, void *cuda_stream)
{
    if (!gate) return HS2_ERR_INVALID_ARG;
    return sparse_decode_impl(hp, Q, K, V, idx, sink, gate, O, LSE, ws, ws_bytes, cuda_stream);
}

static hs2_status sparse_fp8_impl(const hs2_problem *hp, bool decode, const void *Q, const void *K8, const void *V8,
                                  const float *k_scale, const float *v_scale, const int32_t *idx, const float *sink, void *O,
                                  float *LSE, void *cuda_stream)
{
    Params p;
    hs2_status s = sparse_common(hp, Q, K8, V8, idx, O, &p);
    if (s != HS2_OK) return s;
    if (!k_scale || !v_scale) return HS2_ERR_INVALID_ARG;
    if (decode && p.Lq != 1) return HS2_ERR_INVALID_ARG;
    if (!aligned16(Q, K8, V8, O)) return HS2_ERR_UNSUPPORTED;
    Params pm = p;   // the mma.sync kernel's view: a group of 16 as two sub-groups of 8
    split_into_subgroups(&pm, hp->dtype);
    const bool mma = sparse_fp8_supported(pm, hp->dtype);
    // larger head groups and head_dim 256 (the paper's own shape): the tcgen05 gather kernel, dequantising as it gathers
    const bool tc5 = !mma && !g_disable_tc5.load(std::memory_order_relaxed) && sparse_tc5_fp8_supported(p, hp->dtype);
    if (!mma && !tc5) return HS2_ERR_UNSUPPORTED;
    if ((s = check_device()) != HS2_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (mma)
        e = decode ? launch_sparse_fp8_decode(pm, Q, K8, V8, k_scale, v_scale, idx, sink, O, LSE, st)
                   : launch_sparse_fp8_prefill(pm, Q, K8, V8, k_scale, v_scale, idx, sink, O, LSE, st);
    else
        e = launch_sparse_tc5_fp8(p, Q, K8, V8, k_scale, v_scale, idx, sink, O, LSE, nullptr, 0, st);   // no scratch: keys never split
    if (e == cudaErrorNotSupported) {
        (void)cudaGetLastError();
        return HS2_ERR_UNSUPPORTED;
    }
    return e == cudaSuccess ? HS2_OK : cuda_fail(e);
}

hs2_status hs2_sparse_attn_prefill_fp8kv(const hs2_problem *hp, const void *Q, const void *K8, const void *V8,
                                         const float *k_scale, const float *v_scale, const int32_t *idx,
                                         const float *sink, void *O, float *LSE, void *cuda_stream)
{
    return sparse_fp8_impl(hp, false, Q, K8, V8, k_scale, v_scale, idx, sink, O, LSE, cuda_stream);
}

hs2_status hs2_sparse_attn_decode_fp8kv(const hs2_problem *hp, const void *Q, const void *K8, const void *V8,
                                        const float *k_scale, const float *v_scale, const int32_t *idx,
                                        const float *sink, void *O, float *LSE, void *cuda_stream)
{
    return sparse_fp8_impl(hp, true, Q, K8, V8, k_scale, v_scale, idx, sink, O, LSE, cuda_stream);
}

hs2_status hs2_full_attn_select_fp8kv(const hs2_problem *hp, const void *Q, const void *K8, const void *V8,
                                      const float *k_scale, const float *v_scale, void *O, float *LSE, int32_t *idx,
                                      void *ws, size_t ws_bytes, void *cuda_stream)
{
    Params p;
    hs2_status s = resolve(hp, true, &p);
    if (s != HS2_OK) return s;
    if (!Q || !K8 || !V8 || !k_scale || !v_scale || !O || !LSE) return HS2_ERR_INVALID_ARG;
    // One query per sequence only: a prefill-shaped full layer attends to the bf16 K and V it has just produced; it
    // is the decode step that reads the quantised cache.
    if (p.Lq != 1) return HS2_ERR_UNSUPPORTED;
    Params pd = p;   // a sweep over the whole cache: the gather kernel with no index list and a window that covers the context
    pd.k = 0; pd.w = p.Lk;
    if (!aligned16(Q, K8, V8, O) || (int64_t)p.B * p.Hkv > 65535) return HS2_ERR_UNSUPPORTED;
    const bool want_sel = idx != nullptr && p.k > 0;
    if (!sparse_fp8_supported(pd, hp->dtype)) {
        // Larger head groups and head_dim 256 (the paper's own shape): the attention sweeps the cache on the tcgen05
        // gather kernel (the CTAs that split a sequence merge inside a cluster, no scratch), a second pass over the K
        // codes gives the selection scores once the LSE is known, the top-k runs on those rows.
        if (g_disable_tc5.load(std::memory_order_relaxed) || !sparse_tc5_fp8_supported(pd, hp->dtype) || p.blk > 1) return HS2_ERR_UNSUPPORTED;
        const size_t need = want_sel ? align_up((size_t)p.B * p.Hkv * strip_row_bytes(p), 256) : 0;
        if (!ws_ok(ws, ws_bytes, need)) return HS2_ERR_WORKSPACE_TOO_SMALL;
        if ((s = check_device()) != HS2_OK) return s;
        cudaStream_t st2 = (cudaStream_t)cuda_stream;
        cudaError_t e2 = launch_sparse_tc5_fp8(pd, Q, K8, V8, k_scale, v_scale, nullptr, nullptr, O, LSE, nullptr, 0, st2);
        if (e2 == cudaErrorNotSupported) {
            (void)cudaGetLastError();
            return HS2_ERR_UNSUPPORTED;
        }
        if (e2 != cudaSuccess) return cuda_fail(e2);
        if (!want_sel) return HS2_OK;
        float *strip2 = static_cast<float *>(ws);
        const int64_t stride2 = (int64_t)(strip_row_bytes(p) / sizeof(float));
        if ((e2 = launch_scores_fp8_decode(p, Q, K8, k_scale, LSE, strip2, stride2, st2)) != cudaSuccess) return cuda_fail(e2);
        if ((e2 = launch_select(p, strip2, stride2, idx, 0, select_rows(p), st2)) != cudaSuccess) return cuda_fail(e2);
        return HS2_OK;
    }
    const DecodeFusedPlan fu = decode_fused_plan(pd, 0);
    if (want_sel) {
        if (!fu.ok) return HS2_ERR_UNSUPPORTED;   // the raw products of this problem would not fit the scratch cap
        if (!ws_ok(ws, ws_bytes, fu.total)) return HS2_ERR_WORKSPACE_TOO_SMALL;
    }
    if ((s = check_device()) != HS2_OK) return s;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    float *raw = want_sel ? reinterpret_cast<float *>(static_cast<char *>(ws) + fu.off_raw) : nullptr;
    cudaError_t e = launch_sparse_fp8_decode(pd, Q, K8, V8, k_scale, v_scale, nullptr, nullptr, O, LSE, st, raw);
    if (e != cudaSuccess) return cuda_fail(e);
    if (!want_sel) return HS2_OK;
    float *strip = reinterpret_cast<float *>(static_cast<char *>(ws) + fu.off_strip);
    const int64_t stride = (int64_t)(strip_row_bytes(p) / sizeof(float));
    if ((e = launch_scores_from_raw(p, raw, LSE, strip, stride, st)) != cudaSuccess) return cuda_fail(e);
    if ((e = launch_select(p, strip, stride, idx, 0, select_rows(p), st)) != cudaSuccess) return cuda_fail(e);
    return HS2_OK;
}

hs2_status hs2_kv_project(int64_t n_tokens, int32_t d_model, int32_t n_out, const void *H, int64_t ldh, const void *W,
                          int64_t ldw, void *C, int64_t ldc, float *scales, void *cuda_stream)
{
    if (n_tokens < 0 || d_model <= 0 || n_out <= 0 || !H || !W || !C) return HS2_ERR_INVALID_ARG;
    if (n_tokens == 0) return HS2_OK;
    if (!kv_project_supported(n_tokens, n_out, d_model, ldh, ldw, ldc, scales != nullptr) || !aligned16(H, W, C, C))
        return HS2_ERR_UNSUPPORTED;
    hs2_status s = check_device();
    if (s != HS2_OK) return s;
    const cudaError_t e = launch_kv_project(n_tokens, n_out, d_model, H, ldh, W, ldw, C, ldc, scales, (cudaStream_t)cuda_stream);
    if (e == cudaErrorNotSupported) {
        (void)cudaGetLastError();
        return HS2_ERR_UNSUPPORTED;
    }
    return e == cudaSuccess ? HS2_OK : cuda_fail(e);
}

hs2_status hs2_kv_project_fp8_records(int64_t n_tokens, int32_t d_model, int32_t n_out, const void *H, int64_t ldh,
                                      const void *W, int64_t ldw, void *C, int64_t ldc, int64_t ld_group, float *scales,
                                      int64_t scale_ld_token, int64_t scale_ld_group, void *cuda_stream)
{
    if (n_tokens < 0 || d_model <= 0 || n_out <= 0 || !H || !W || !C || !scales) return HS2_ERR_INVALID_ARG;
    if (ld_group < 128 || scale_ld_token < 0 || scale_ld_group < 0) return HS2_ERR_INVALID_ARG;
    if (n_tokens == 0) return HS2_OK;
    // (the row stride only has to hold what a token's groups span, not n_out packed bytes)
    if (!kv_project_supported(n_tokens, n_out, d_model, ldh, ldw, (int64_t)n_out, true) || ldc % 16 != 0 || ld_group % 16 != 0 ||
        ldc < (n_out / 128 - 1) * ld_group + 128 || !aligned16(H, W, C, C) || (reinterpret_cast<uintptr_t>(scales) & 3u))
        return HS2_ERR_UNSUPPORTED;
    hs2_status s = check_device();
    if (s != HS2_OK) return s;
    const cudaError_t e = launch_kv_project_records(n_tokens, n_out, d_model, H, ldh, W, ldw, C, ldc, ld_group, scales,
                                                    scale_ld_token, scale_ld_group, (cudaStream_t)cuda_stream);
    if (e == cudaErrorNotSupported) {
        (void)cudaGetLastError();
        return HS2_ERR_UNSUPPORTED;
    }
    return e == cudaSuccess ? HS2_OK : cuda_fail(e);
}

hs2_status hs2_sparse_attn_decode_static(const hs2_problem *hp, const void *Q, const void *K, const void *V,
                                         const int32_t *idx, const float *sink, void *O, float *LSE,
                                         void *cuda_stream)
{
    Params p;
    hs2_status s = sparse_common(hp, Q, K, V, idx, O, &p);
    if (s != HS2_OK) return s;
    if (p.Lq != 1) return HS2_ERR_INVALID_ARG;
    split_into_subgroups(&p, hp->dtype);
    if (!(sparse_mma_supported(p, hp->dtype) && aligned16(Q, K, V, O))) return HS2_ERR_UNSUPPORTED;
    if (!sparse_mma_decode_static_fits(p)) return HS2_ERR_STATIC_SCRATCH;
    if ((s = check_device()) != HS2_OK) return s;
    cudaError_t e = launch_sparse_mma_decode_static(p, Q, K, V, idx, sink, O, LSE, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? HS2_OK : cuda_fail(e);
}

hs2_status hs2_probe_gather(const hs2_problem *hp, const void *K, const void *V, const int32_t *idx, int mode,
                            unsigned *sink_word, void *cuda_stream)
{
    Params p;
    hs2_status s = resolve(hp, true, &p);
    if (s != HS2_OK) return s;
    if (!K || !V || !sink_word || (p.k > 0 && !idx) || (mode != 0 && mode != 1)) return HS2_ERR_INVALID_ARG;
    if (hp->dtype != HS2_BF16 || p.D != 128 || p.ks_t % 8 || p.ks_h % 8 || p.ks_b % 8 ||
        (reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V)) % 16)
        return HS2_ERR_UNSUPPORTED;
    if ((s = check_device()) != HS2_OK) return s;
    const cudaError_t e = launch_probe_gather(p, K, V, idx, mode, sink_word, (cudaStream_t)cuda_stream);
    if (e == cudaErrorNotSupported) {
        (void)cudaGetLastError();
        return HS2_ERR_UNSUPPORTED;
    }
    return e == cudaSuccess ? HS2_OK : cuda_fail(e);
}

const char *hs2_status_string(hs2_status s)
{
    switch (s) {
        case HS2_OK: return "ok";
        case HS2_ERR_INVALID_ARG: return "invalid argument";
        case HS2_ERR_UNSUPPORTED: return "unsupported problem";
        case HS2_ERR_WORKSPACE_TOO_SMALL: return "workspace too small or misaligned";
        case HS2_ERR_CUDA: return "CUDA runtime error";
        case HS2_ERR_STATIC_SCRATCH: return "problem needs more scratch than the library's built-in array holds";
    }
    return "unknown status";
}

int hs2_last_cuda_error(void) { return g_last_cuda_error; }

int hs2_device_error_flags(unsigned *flags)
{
    if (!flags) return HS2_ERR_INVALID_ARG;
    unsigned a = 0, b = 0, c = 0, d = 0;
    cudaError_t e = read_tc5_error(&a);
    if (e == cudaSuccess) e = read_sparse_error(&b);
    if (e == cudaSuccess) e = read_sparse_tc5_error(&c);
    if (e == cudaSuccess) e = read_kvproj_error(&d);
    *flags = a | (b << 8) | (c << 16) | (d << 24);   // bits 8.. : the mma.sync sparse kernels, bits 16.. : the tcgen05 sparse kernel, bits 24.. : the KV projection
    return e == cudaSuccess ? HS2_OK : cuda_fail(e);
}

int hs2_set_tcgen05_enabled(int enabled)
{
    const int old = g_disable_tc5.load(std::memory_order_relaxed) ? 0 : 1;
    if (enabled >= 0) g_disable_tc5.store(enabled ? 0 : 1, std::memory_order_relaxed);
    return old;
}

int hs2_set_filter_min_keys(int min_keys)
{
    const int old = g_filter_min_keys.load(std::memory_order_relaxed);
    if (min_keys > 0) g_filter_min_keys.store(min_keys, std::memory_order_relaxed);
    return old;
}

unsigned long long hs2_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
