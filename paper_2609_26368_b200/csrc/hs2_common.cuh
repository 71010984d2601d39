// Internal declarations shared by the hs2 translation units (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hs2.h"

namespace hs2 {

// A validated problem with every default resolved; passed to kernels by value.
struct Params {
    int B, Hq, Hkv, G, D;
    int Lq, Lk;
    int k, w;
    float scale;        // softmax scale
    float scale_log2;   // scale * log2(e): logits are kept in the base-2 domain inside the kernels
    const int32_t *q_start;
    const int32_t *kv_lens;
    int64_t qs_b, qs_t, qs_h;   // element strides
    int64_t ks_b, ks_t, ks_h;
    int64_t os_b, os_t, os_h;
    int64_t ss_b, ss_t, ss_h;   // FP8 cache: strides of the scale arrays, in floats
    int share;          // > 1: consecutive groups of `share` KV-head slots are one real KV head seen through sub-groups
                        // of its query heads (K, V and idx are indexed by slot / share); 0 or 1: plain
    int blk;            // selection granularity: 1 = tokens, B > 1 = aligned blocks of B tokens
    const void *gate;   // optional output-gate logits of the sparse layers: shape, dtype and strides of O; null = no gate
};

// sigmoid output gate of the sparse layers (Section 4.1): the attention output is multiplied elementwise by
// sigmoid(gate logit)
__device__ __forceinline__ float gate_of(float logit) { return 1.f / (1.f + __expf(-logit)); }

// per-sequence geometry, clamped so that no later index arithmetic can leave the tensors
__device__ __forceinline__ int kvlen_of(const Params &p, int b)
{
    int n = p.kv_lens ? p.kv_lens[b] : p.Lk;
    return n < 0 ? 0 : (n > p.Lk ? p.Lk : n);
}
__device__ __forceinline__ int pos_of(const Params &p, int b, int i)
{
    const int kvl = p.kv_lens ? p.kv_lens[b] : p.Lk;
    const int q0 = p.q_start ? p.q_start[b] : kvl - p.Lq;
    return q0 + i;
}

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float &dst, float x) { dst = x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16 &dst, float x) { dst = __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// every kernel launch of the library is counted here (read through hs2_launch_count)
void count_launch(int n = 1);

// ---- launchers (one per translation unit); each returns the cudaError_t of its launches ----

// Generic SIMT kernels: fp32 arithmetic on fp32 or bf16 tensors, any head_dim <= 256, any group size.
cudaError_t launch_full_attn_generic(const Params &p, hs2_dtype dt, const void *Q, const void *K, const void *V,
                                     void *O, float *LSE, cudaStream_t st);
// Group scores a[j] for rows [row0, row0+n_rows) of the flattened (b, g, i) index into `out`
// (row stride out_stride).  all_visible: also write window keys and -inf beyond the causal limit.
cudaError_t launch_scores_generic(const Params &p, hs2_dtype dt, const void *Q, const void *K, const float *LSE,
                                  float *out, int64_t out_stride, int64_t row0, int64_t n_rows, bool all_visible,
                                  cudaStream_t st);
cudaError_t launch_sparse_generic(const Params &p, hs2_dtype dt, const void *Q, const void *K, const void *V,
                                  const int32_t *idx, const float *sink, void *O, float *LSE, cudaStream_t st);

// Block-level selection (p.blk > 1) over score rows [row0, row0+n_rows); `scores` points at row row0.
cudaError_t launch_block_select(const Params &p, const float *scores, int64_t score_stride, int32_t *idx, int64_t row0,
                                int64_t n_rows, cudaStream_t st);
// Radix select over score rows [row0, row0+n_rows); `scores` points at row row0.
cudaError_t launch_topk(const Params &p, const float *scores, int64_t score_stride, int32_t *idx,
                        int64_t row0, int64_t n_rows, cudaStream_t st);

// Filtered selection: thresholds from sampled strips, selection from candidate lists, exact redo of flagged rows.
int filter_sample_width(const Params &p, int samp);
cudaError_t launch_filter_thresholds(const Params &p, const float *sample, int64_t stride, int64_t row0, int64_t n_rows,
                                     int samp, int cap, uint32_t *tau_key, int *flag, cudaStream_t st);
cudaError_t launch_filter_select(const Params &p, const void *cand, const int *count, int cap,
                                 int32_t *idx, int64_t row0, int64_t n_rows, int *flag, cudaStream_t st);
cudaError_t launch_select_recompute(const Params &p, const void *Q, const void *K, const float *LSE, int32_t *idx,
                                    int64_t row0, int64_t n_rows, const int *flag, cudaStream_t st);

// Tensor-core bf16 kernels (head_dim 128, group <= 8).
bool sparse_mma_supported(const Params &p, hs2_dtype dt);
cudaError_t launch_sparse_mma_prefill(const Params &p, const void *Q, const void *K, const void *V, const int32_t *idx,
                                      const float *sink, void *O, float *LSE, cudaStream_t st);
size_t sparse_mma_decode_ws_bytes(const Params &p);
// raw (optional): float [B * Hkv][G][Lk]; receives the unscaled q.k of every attended (head, key)
cudaError_t launch_sparse_mma_decode(const Params &p, const void *Q, const void *K, const void *V, const int32_t *idx,
                                     const float *sink, void *O, float *LSE, void *ws, size_t ws_bytes,
                                     cudaStream_t st, float *raw = nullptr);
// group scores of a single-query layer from those raw products (rows = (b, g), row stride out_stride)
cudaError_t launch_scores_from_raw(const Params &p, const float *raw, const float *LSE, float *out, int64_t out_stride,
                                   cudaStream_t st);

// Decode with the partials in a static device array of the library (no caller scratch).
constexpr int kStaticDecodeMaxPairs = HS2_STATIC_DECODE_MAX_PAIRS;
bool sparse_mma_decode_static_fits(const Params &p);
cudaError_t launch_sparse_mma_decode_static(const Params &p, const void *Q, const void *K, const void *V,
                                            const int32_t *idx, const float *sink, void *O, float *LSE, cudaStream_t st);

bool full_mma_supported(const Params &p, hs2_dtype dt);
cudaError_t launch_full_attn_mma(const Params &p, const void *Q, const void *K, const void *V, void *O, float *LSE,
                                 cudaStream_t st);
cudaError_t launch_scores_mma(const Params &p, const void *Q, const void *K, const float *LSE, float *out,
                              int64_t out_stride, int64_t row0, int64_t n_rows, bool all_visible, cudaStream_t st);

// tcgen05 / TMEM / TMA full attention (bf16, head_dim 128)
bool full_tc5_supported(const Params &p, hs2_dtype dt);        // head_dim 128: attention, score sweeps, filters
bool full_attn_tc5_supported(const Params &p, hs2_dtype dt);   // the attention kernel alone: head_dim 128 or 256
cudaError_t launch_full_attn_tc5(const Params &p, const void *Q, const void *K, const void *V, void *O, float *LSE,
                                 cudaStream_t st);
bool scores_tc5_supported(const Params &p, hs2_dtype dt);
cudaError_t launch_scores_tc5(const Params &p, const void *Q, const void *K, const float *LSE, float *out,
                              int64_t out_stride, int64_t row0, int64_t n_rows, bool all_visible, cudaStream_t st);
bool scores_filter_supported(const Params &p, hs2_dtype dt);
cudaError_t launch_scores_sampled_tc5(const Params &p, const void *Q, const void *K, const float *LSE, float *out,
                                      int64_t out_stride, int64_t row0, int64_t n_rows, int samp, cudaStream_t st);
cudaError_t launch_scores_filter_tc5(const Params &p, const void *Q, const void *K, const float *LSE, int64_t row0,
                                     int64_t n_rows, const uint32_t *tau_key, void *cand, int *count,
                                     int cap, cudaStream_t st);
// tcgen05 sparse attention for large head groups (bf16, head_dim 128 or 256, 8 < group <= 128)
bool sparse_tc5_supported_shape(const Params &p, hs2_dtype dt);   // the shape alone (no driver query)
bool sparse_tc5_supported(const Params &p, hs2_dtype dt);
size_t sparse_tc5_ws_bytes(const Params &p);   // scratch that lets few queries (decode) split their keys over CTAs
cudaError_t launch_sparse_tc5(const Params &p, const void *Q, const void *K, const void *V, const int32_t *idx,
                              const float *sink, void *O, float *LSE, void *ws, size_t ws_bytes, cudaStream_t st);
// the same kernel on an e4m3 cache with per-(token, KV head) scales (bf16 queries; any group up to 128, head_dim 128 or 256)
bool sparse_tc5_fp8_supported(const Params &p, hs2_dtype dt);
cudaError_t launch_sparse_tc5_fp8(const Params &p, const void *Q, const void *K8, const void *V8, const float *ksc,
                                  const float *vsc, const int32_t *idx, const float *sink, void *O, float *LSE, void *ws,
                                  size_t ws_bytes, cudaStream_t st);
cudaError_t read_sparse_tc5_error(unsigned *out);
// FP8 (e4m3 + per-(token, KV head) scale) KV cache, bf16 queries: head_dim 128, group <= 8
bool sparse_fp8_supported(const Params &p, hs2_dtype dt);
cudaError_t launch_sparse_fp8_prefill(const Params &p, const void *Q, const void *K, const void *V, const float *ksc,
                                      const float *vsc, const int32_t *idx, const float *sink, void *O, float *LSE,
                                      cudaStream_t st);
cudaError_t launch_sparse_fp8_decode(const Params &p, const void *Q, const void *K, const void *V, const float *ksc,
                                     const float *vsc, const int32_t *idx, const float *sink, void *O, float *LSE,
                                     cudaStream_t st, float *raw = nullptr);
// selection scores of a one-query layer on the FP8 cache (any group up to 128, head_dim 128 or 256), rows = (b, g)
cudaError_t launch_scores_fp8_decode(const Params &p, const void *Q, const void *K8, const float *ksc, const float *LSE,
                                     float *out, int64_t out_stride, cudaStream_t st);
// KV-cache producer: C[T, N] = H[T, dm] W[N, dm]^T, bf16 out or e4m3 codes + scale per (token, 128 columns)
bool kv_project_supported(int64_t T, int N, int dm, int64_t ldh, int64_t ldw, int64_t ldc, bool fp8);
cudaError_t launch_kv_project(int64_t T, int N, int dm, const void *H, int64_t ldh, const void *W, int64_t ldw, void *C,
                              int64_t ldc, float *scales, cudaStream_t st);
// the e4m3 output with a stride between the 128-column groups and strided scales (records that hold codes and scales)
cudaError_t launch_kv_project_records(int64_t T, int N, int dm, const void *H, int64_t ldh, const void *W, int64_t ldw,
                                      void *C, int64_t ldc, int64_t ld_group, float *scales, int64_t s_tok, int64_t s_grp,
                                      cudaStream_t st);
cudaError_t read_kvproj_error(unsigned *out);
// the row fetches of the sparse prefill and nothing else (measurement aid); mode 0: L2 loads, 1: through L1
cudaError_t launch_probe_gather(const Params &p, const void *K, const void *V, const int32_t *idx, int mode,
                                unsigned *out, cudaStream_t st);
cudaError_t read_tc5_error(unsigned *out);
cudaError_t read_sparse_error(unsigned *out);

}  // namespace hs2
