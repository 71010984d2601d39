// Generic SIMT kernels: fp32 arithmetic on fp32 or bf16 tensors, any head_dim <= 256 and any
// GQA group size.  They are the fp32 path (where a bf16 tensor-core product would break the 1e-4
// tolerance) and the path for shapes the tensor-core kernels do not cover.
//
// One warp owns one output row.  Keys are taken 32 at a time: lane t scores key t (a dot product
// over head_dim), the warp does the online-softmax bookkeeping with shuffles, then the lanes switch
// to owning output dimensions (d = lane, lane+32, ...) and accumulate P.V with coalesced V reads.
#include "hs2_common.cuh"

namespace hs2 {
namespace {

constexpr int kWarpsPerBlock = 4;
constexpr int kMaxDPerLane = 8;   // head_dim <= 256

template <typename T> struct Vec;
template <> struct Vec<float> { static constexpr int n = 4; using type = float4; };
template <> struct Vec<__nv_bfloat16> { static constexpr int n = 8; using type = uint4; };

__device__ __forceinline__ void unpack(const float4 &v, float *f) { f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w; }
__device__ __forceinline__ void unpack(const uint4 &v, float *f)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// <q, k_row> with q in shared memory (fp32) and the key row in global memory
template <typename T>
__device__ __forceinline__ float dot_row(const float *sq, const T *krow, int D, bool vec_ok)
{
    float acc = 0.f;
    if (vec_ok) {
        constexpr int N = Vec<T>::n;
        const typename Vec<T>::type *kv = reinterpret_cast<const typename Vec<T>::type *>(krow);
        for (int d = 0; d < D; d += N) {
            float f[N];
            unpack(__ldg(kv + d / N), f);
#pragma unroll
            for (int e = 0; e < N; ++e) acc = fmaf(f[e], sq[d + e], acc);
        }
    } else {
        for (int d = 0; d < D; ++d) acc = fmaf(to_f32(krow[d]), sq[d], acc);
    }
    return acc;
}

template <typename T>
__device__ __forceinline__ bool vec_ok_for(const Params &p, const void *K)
{
    constexpr int N = Vec<T>::n;
    return (p.D % N == 0) && (p.ks_b % N == 0) && (p.ks_t % N == 0) && (p.ks_h % N == 0) &&
           (reinterpret_cast<uintptr_t>(K) % 16 == 0);
}

// Online-softmax state of one row, distributed over a warp: m, l replicated; acc[r] is output
// dimension lane + 32 r.
struct RowState {
    float m, l;
    float acc[kMaxDPerLane];
};

// Fold one chunk of up to 32 keys into the state.  t2 = this lane's scaled logit in the base-2
// domain (-inf when the lane has no key); vrow(t) gives the V row of lane t's key.
template <typename T, typename VRow>
__device__ __forceinline__ void fold_chunk(RowState &st, float t2, unsigned valid_mask, int D, int lane, VRow vrow)
{
    const float mc = warp_max(t2);
    const float m_new = fmaxf(st.m, mc);
    if (m_new == -INFINITY) return;   // nothing finite yet
    const float corr = exp2f(st.m - m_new);
    const float pj = exp2f(t2 - m_new);   // 0 for -inf
    st.l = st.l * corr + warp_sum(pj);
    st.m = m_new;
#pragma unroll
    for (int r = 0; r < kMaxDPerLane; ++r) st.acc[r] *= corr;
    unsigned mask = valid_mask;
    while (mask) {
        const int t = __ffs(mask) - 1;
        mask &= mask - 1;
        const float pt = __shfl_sync(0xffffffffu, pj, t);
        const T *v = vrow(t);
#pragma unroll
        for (int r = 0; r < kMaxDPerLane; ++r) {
            const int d = lane + 32 * r;
            if (d < D) st.acc[r] = fmaf(pt, to_f32(v[d]), st.acc[r]);
        }
    }
}

template <typename T>
__device__ __forceinline__ void write_row(const RowState &st, T *o, float *lse_out, int D, int lane, const T *gate = nullptr)
{
    const float inv = st.l > 0.f ? 1.f / st.l : 0.f;
#pragma unroll
    for (int r = 0; r < kMaxDPerLane; ++r) {
        const int d = lane + 32 * r;
        if (d < D) from_f32(o[d], st.acc[r] * inv * (gate ? gate_of(to_f32(gate[d])) : 1.f));
    }
    if (lse_out && lane == 0) *lse_out = st.l > 0.f ? (st.m + log2f(st.l)) * kLn2 : -INFINITY;
}

// ---------------------------------------------------------------- full causal attention
template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
k_full_generic(const Params p, const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
               T *__restrict__ O, float *__restrict__ LSE)
{
    extern __shared__ float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * kWarpsPerBlock + warp;   // (b, h, i), i fastest
    if (row >= (int64_t)p.B * p.Hq * p.Lq) return;
    const int i = (int)(row % p.Lq);
    const int h = (int)((row / p.Lq) % p.Hq);
    const int b = (int)(row / ((int64_t)p.Lq * p.Hq));
    const int g = h / p.G;
    float *sq = smem + warp * p.D;
    const T *q = Q + b * p.qs_b + i * p.qs_t + h * p.qs_h;
    for (int d = lane; d < p.D; d += 32) sq[d] = to_f32(q[d]);
    __syncwarp();
    const int kvl = kvlen_of(p, b);
    const int pos = pos_of(p, b, i);
    const int n = min(pos + 1, kvl);   // visible keys 0..n-1
    const T *kb = K + b * p.ks_b + g * p.ks_h;
    const T *vb = V + b * p.ks_b + g * p.ks_h;
    const bool vec_ok = vec_ok_for<T>(p, K);
    RowState st;
    st.m = -INFINITY; st.l = 0.f;
#pragma unroll
    for (int r = 0; r < kMaxDPerLane; ++r) st.acc[r] = 0.f;
    for (int c = 0; c < n; c += 32) {
        const int j = c + lane;
        const bool valid = j < n;
        const float t2 = valid ? dot_row<T>(sq, kb + (int64_t)j * p.ks_t, p.D, vec_ok) * p.scale_log2 : -INFINITY;
        const unsigned mask = __ballot_sync(0xffffffffu, valid);
        fold_chunk<T>(st, t2, mask, p.D, lane, [&](int t) { return vb + (int64_t)(c + t) * p.ks_t; });
    }
    write_row<T>(st, O + b * p.os_b + i * p.os_t + h * p.os_h, LSE + row, p.D, lane);
}

// ---------------------------------------------------------------- group selection scores
// a[j] = max over the heads h of group g of (scale <q_h, k_j> - LSE_h); one warp per (b, g, i) row.
template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
k_scores_generic(const Params p, const T *__restrict__ Q, const T *__restrict__ K, const float *__restrict__ LSE,
                 float *__restrict__ out, int64_t out_stride, int64_t row0, int64_t n_rows, int all_visible)
{
    extern __shared__ float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t lr = (int64_t)blockIdx.x * (blockDim.x >> 5) + warp;   // the launcher sizes the block to the shared memory
    if (lr >= n_rows) return;
    const int64_t row = row0 + lr;   // (b, g, i), i fastest
    const int i = (int)(row % p.Lq);
    const int g = (int)((row / p.Lq) % p.Hkv);
    const int b = (int)(row / ((int64_t)p.Lq * p.Hkv));
    float *sq = smem + (size_t)warp * p.G * p.D;
    for (int e = lane; e < p.G * p.D; e += 32) {
        const int hh = e / p.D, d = e % p.D;
        sq[e] = to_f32(Q[b * p.qs_b + i * p.qs_t + (g * p.G + hh) * p.qs_h + d]);
    }
    __syncwarp();
    const int kvl = kvlen_of(p, b);
    const int pos = pos_of(p, b, i);
    const int n_vis = max(0, min(pos + 1, kvl));
    const int n_cand = max(0, min(pos - p.w + 1, kvl));
    const int n = all_visible ? n_vis : n_cand;
    const T *kb = K + b * p.ks_b + g * p.ks_h;
    const bool vec_ok = vec_ok_for<T>(p, K);
    float *orow = out + lr * out_stride;
    const float *lse = LSE + ((int64_t)b * p.Hq + g * p.G) * p.Lq + i;   // + hh * Lq
    for (int c = 0; c < n; c += 32) {
        const int j = c + lane;
        if (j < n) {
            float a = -INFINITY;
            for (int hh = 0; hh < p.G; ++hh) {
                const float s = dot_row<T>(sq + hh * p.D, kb + (int64_t)j * p.ks_t, p.D, vec_ok);
                a = fmaxf(a, fmaf(s, p.scale, -lse[(int64_t)hh * p.Lq]));
            }
            orow[j] = a;
        }
    }
    if (all_visible)
        for (int j = n + lane; j < p.Lk; j += 32) orow[j] = -INFINITY;
}

// ---------------------------------------------------------------- sparse attention (prefill and decode)
// Attended set of query (b, i) for KV head g: valid entries of idx row (b, g, i) plus the window.
template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
k_sparse_generic(const Params p, const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                 const int32_t *__restrict__ idx, const float *__restrict__ sink, T *__restrict__ O,
                 float *__restrict__ LSE)
{
    extern __shared__ float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * kWarpsPerBlock + warp;   // (b, h, i), i fastest
    if (row >= (int64_t)p.B * p.Hq * p.Lq) return;
    const int i = (int)(row % p.Lq);
    const int h = (int)((row / p.Lq) % p.Hq);
    const int b = (int)(row / ((int64_t)p.Lq * p.Hq));
    const int g = h / p.G;
    float *sq = smem + warp * p.D;
    const T *q = Q + b * p.qs_b + i * p.qs_t + h * p.qs_h;
    for (int d = lane; d < p.D; d += 32) sq[d] = to_f32(q[d]);
    __syncwarp();
    const int kvl = kvlen_of(p, b);
    const int pos = pos_of(p, b, i);
    const T *kb = K + b * p.ks_b + g * p.ks_h;
    const T *vb = V + b * p.ks_b + g * p.ks_h;
    const int32_t *irow = idx + (((int64_t)b * p.Hkv + g) * p.Lq + i) * p.k;
    const bool vec_ok = vec_ok_for<T>(p, K);
    RowState st;
    st.m = sink ? sink[h] * kLog2e : -INFINITY;
    st.l = sink ? (st.m == -INFINITY ? 0.f : 1.f) : 0.f;
#pragma unroll
    for (int r = 0; r < kMaxDPerLane; ++r) st.acc[r] = 0.f;
    const int n_slots = p.k + p.w;
    for (int c = 0; c < n_slots; c += 32) {
        const int s = c + lane;
        int j = -1;
        bool valid = false;
        if (s < p.k) {
            j = irow[s];
            valid = j >= 0 && j <= pos - p.w && j < kvl;
        } else if (s < n_slots) {
            j = pos - p.w + 1 + (s - p.k);
            valid = j >= 0 && j <= pos && j < kvl;
        }
        const unsigned mask = __ballot_sync(0xffffffffu, valid);
        if (mask == 0) continue;
        const float t2 = valid ? dot_row<T>(sq, kb + (int64_t)j * p.ks_t, p.D, vec_ok) * p.scale_log2 : -INFINITY;
        fold_chunk<T>(st, t2, mask, p.D, lane, [&](int t) {
            const int jt = __shfl_sync(0xffffffffu, j, t);
            return vb + (int64_t)jt * p.ks_t;
        });
    }
    const int64_t o_off = b * p.os_b + i * p.os_t + h * p.os_h;
    write_row<T>(st, O + o_off, LSE ? LSE + row : nullptr, p.D, lane, p.gate ? static_cast<const T *>(p.gate) + o_off : nullptr);
}

template <typename Kern>
cudaError_t set_smem(Kern kern, size_t bytes)
{
    if (bytes > 48 * 1024) return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    return cudaSuccess;
}

}  // namespace

cudaError_t launch_full_attn_generic(const Params &p, hs2_dtype dt, const void *Q, const void *K, const void *V,
                                     void *O, float *LSE, cudaStream_t st)
{
    const int64_t rows = (int64_t)p.B * p.Hq * p.Lq;
    if (rows == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((rows + kWarpsPerBlock - 1) / kWarpsPerBlock);
    const size_t smem = sizeof(float) * kWarpsPerBlock * p.D;
    if (dt == HS2_F32)
        k_full_generic<float><<<blocks, kWarpsPerBlock * 32, smem, st>>>(p, (const float *)Q, (const float *)K,
                                                                          (const float *)V, (float *)O, LSE);
    else
        k_full_generic<__nv_bfloat16><<<blocks, kWarpsPerBlock * 32, smem, st>>>(
            p, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, (__nv_bfloat16 *)O, LSE);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_scores_generic(const Params &p, hs2_dtype dt, const void *Q, const void *K, const float *LSE,
                                  float *out, int64_t out_stride, int64_t row0, int64_t n_rows, bool all_visible,
                                  cudaStream_t st)
{
    if (n_rows == 0) return cudaSuccess;
    // each warp keeps the G query vectors of its row in shared memory: fewer warps per block for large groups
    const size_t per_warp = sizeof(float) * (size_t)p.G * p.D;
    int warps = (int)((200 * 1024) / per_warp);
    warps = warps < 1 ? 1 : (warps > kWarpsPerBlock ? kWarpsPerBlock : warps);
    if (per_warp > 227 * 1024) return cudaErrorInvalidConfiguration;
    const unsigned blocks = (unsigned)((n_rows + warps - 1) / warps);
    const size_t smem = per_warp * warps;
    cudaError_t e;
    if (dt == HS2_F32) {
        if ((e = set_smem(k_scores_generic<float>, smem)) != cudaSuccess) return e;
        k_scores_generic<float><<<blocks, warps * 32, smem, st>>>(p, (const float *)Q, (const float *)K, LSE, out, out_stride,
                                                                  row0, n_rows, all_visible);
    } else {
        if ((e = set_smem(k_scores_generic<__nv_bfloat16>, smem)) != cudaSuccess) return e;
        k_scores_generic<__nv_bfloat16><<<blocks, warps * 32, smem, st>>>(
            p, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)K, LSE, out, out_stride, row0, n_rows, all_visible);
    }
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_sparse_generic(const Params &p, hs2_dtype dt, const void *Q, const void *K, const void *V,
                                  const int32_t *idx, const float *sink, void *O, float *LSE, cudaStream_t st)
{
    const int64_t rows = (int64_t)p.B * p.Hq * p.Lq;
    if (rows == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((rows + kWarpsPerBlock - 1) / kWarpsPerBlock);
    const size_t smem = sizeof(float) * kWarpsPerBlock * p.D;
    if (dt == HS2_F32)
        k_sparse_generic<float><<<blocks, kWarpsPerBlock * 32, smem, st>>>(
            p, (const float *)Q, (const float *)K, (const float *)V, idx, sink, (float *)O, LSE);
    else
        k_sparse_generic<__nv_bfloat16><<<blocks, kWarpsPerBlock * 32, smem, st>>>(
            p, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)K, (const __nv_bfloat16 *)V, idx, sink,
            (__nv_bfloat16 *)O, LSE);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hs2
