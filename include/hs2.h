/*
 * hs2 — hybrid sparse attention hot path of HySparse2 on B200 (sm_100a).  C ABI.
 *
 * One hybrid block of the paper is a full-attention (FA) layer followed by sparse-attention
 * (SA) layers that reuse the FA layer's KV cache and its token-level selection indices
 * (Section 3.3, "Cross-Layer KV Reuse"; Figure 2, right).  The library covers the attention
 * operators of that block:
 *
 *   hs2_full_attn_select     FA layer: causal softmax attention, which also emits, per query token
 *                            and per KV head, the indices of the k highest-scoring tokens outside
 *                            the forced local window (Sections 3.3 and 3.4).
 *   hs2_topk_select          the same token-level top-k on a score tensor the caller provides.
 *   hs2_sparse_attn_prefill  SA layer: attention over (reused indices) U (forced window of the most
 *                            recent w tokens), K/V read from the FA layer's cache (Section 3.3).
 *   hs2_sparse_attn_decode   the SA layer for one new token per sequence (split over the KV set).
 *   ..._gated                the two SA calls with the sigmoid output gate of the sparse layers fused in.
 *   ..._fp8kv                the two SA calls on an e4m3 KV cache with per-token scales.
 *   hs2_kv_project           the producer of those caches: the K/V projection of KV Bridging (Section 3.2),
 *                            bf16 or quantised to the e4m3 cache format in its epilogue
 *                            (hs2_kv_project_fp8_records: codes and scales into one record per token and KV head).
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller; `hs2_problem` itself is a
 *     host struct read during the call.  `q_start` / `kv_lens` inside it are device arrays.
 *   - Layouts: Q, O  [batch, q_len, n_q_heads, head_dim]; K, V [batch, kv_len, n_kv_heads, head_dim]
 *     (token major; last dimension contiguous; strides in elements, 0 = packed);
 *     idx [batch, n_kv_heads, q_len, k_sel] int32, packed; LSE [batch, n_q_heads, q_len] float, packed.
 *   - Query head h reads KV head h / (n_q_heads / n_kv_heads).  No positional encoding is applied
 *     (Section 4.1: full and sparse attention use NoPE).
 *   - Query i of sequence b sits at absolute position pos = q_start[b] + i and sees keys
 *     0 .. min(pos, kv_lens[b]-1).  The forced window is [pos-w+1, pos] (the token itself counts);
 *     selection candidates are keys 0 .. pos-w.
 *   - The library allocates no memory, enqueues its work on the given CUDA stream and returns
 *     without synchronising.  Scratch comes from the caller (`ws`, at least hs2_workspace_bytes()
 *     bytes, 256-byte aligned).  No result of one call depends on an earlier call; what the process
 *     does keep is listed at the end of this file: two dispatch knobs (hs2_set_tcgen05_enabled,
 *     hs2_set_filter_min_keys), per-device caches of device attributes, a sticky device error word,
 *     a launch counter, and the built-in scratch array of hs2_sparse_attn_decode_static.
 *   - Argument errors are found on the host before anything is launched and reported through the
 *     status; nothing throws, aborts or traps.  There is no CPU fallback: without a CUDA device
 *     every compute entry point returns HS2_ERR_CUDA.
 */
#ifndef HS2_H_
#define HS2_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HS2_OK = 0,
    HS2_ERR_INVALID_ARG = 1,         /* NULL where a pointer is required, non-positive size, bad head ratio ... */
    HS2_ERR_UNSUPPORTED = 2,         /* valid problem outside what the kernels cover (e.g. head_dim > 256) */
    HS2_ERR_WORKSPACE_TOO_SMALL = 3, /* ws_bytes < hs2_workspace_bytes() or ws not 256-byte aligned */
    HS2_ERR_CUDA = 4,                /* a CUDA runtime call failed; see hs2_last_cuda_error() */
    HS2_ERR_STATIC_SCRATCH = 5       /* the problem needs more scratch than the library's built-in array holds */
} hs2_status;

typedef enum { HS2_F32 = 0, HS2_BF16 = 1 } hs2_dtype;

typedef enum {
    HS2_OP_FULL_ATTN_SELECT = 0,
    HS2_OP_TOPK_SELECT = 1,
    HS2_OP_SPARSE_ATTN_PREFILL = 2,
    HS2_OP_SPARSE_ATTN_DECODE = 3,
    HS2_OP_FULL_ATTN_SELECT_FP8KV = 4
} hs2_op;

typedef struct {
    int32_t batch;
    int32_t n_q_heads, n_kv_heads;   /* n_q_heads % n_kv_heads == 0 (GQA; MQA when n_kv_heads == 1) */
    int32_t head_dim;                /* 1..256; K and V share it */
    int32_t q_len, kv_len;           /* tensor extents in tokens */
    int32_t k_sel;                   /* k: tokens selected outside the window (Section 4.1 uses 1024) */
    int32_t window;                  /* w: forced most-recent tokens, the query's own included (paper: 128) */
    float softmax_scale;             /* 0 => 1/sqrt(head_dim) */
    hs2_dtype dtype;                 /* element type of Q, K, V, O */
    const int32_t *q_start;          /* device [batch] or NULL => kv_lens[b] - q_len */
    const int32_t *kv_lens;          /* device [batch] or NULL => kv_len */
    int64_t q_stride[3];             /* elements: (batch, token, head); all 0 => packed */
    int64_t kv_stride[3];            /* shared by K and V */
    int64_t o_stride[3];
    int32_t select_block;            /* selection granularity of hs2_full_attn_select / hs2_topk_select: 0 or 1 =
                                        individual tokens (the paper's method); B > 1 = aligned blocks of B tokens,
                                        the block-level variant the paper ablates against (Section 5, Ablation 1:
                                        block size 64, 1024 tokens = 16 blocks); k_sel must then be a multiple of B */
    int64_t kv_scale_stride[3];      /* FP8 cache entry points only: floats between the scales of consecutive
                                        (batch, token, KV head) entries, shared by the K and the V scales; all 0 =>
                                        packed [batch, kv_len, n_kv_heads].  With kv_stride this lets a cache keep the K
                                        codes, the V codes and both scales of a (token, KV head) in one record */
} hs2_problem;

/* Bytes of scratch `op` needs for this problem (a host-side computation; 0 is a valid answer).
 * Returns 0 for an invalid problem. */
size_t hs2_workspace_bytes(const hs2_problem *p, hs2_op op);

/*
 * FA layer of a hybrid block (Section 3.4: the full-attention layers are the indexers, their own exact
 * attention scores rank the tokens; Section 3.3: top-k over individual tokens, outside the forced window).
 *
 *   O    out  attention output, same layout/dtype as Q
 *   LSE  out  log-sum-exp of the scaled logits per (batch, head, query), natural log; required
 *   (With p->select_block = B > 1 the selection is block-level instead: the candidates of a row are cut into
 *   aligned blocks [B m, B m + B); a block's score is the maximum a[j] over its candidate keys; the k_sel / B
 *   best blocks (ties: lower block first) are kept and idx holds their candidate keys, ascending, -1 padded.)
 *   idx  out  [batch, n_kv_heads, q_len, k_sel] or NULL to skip the selection.  Row (b,g,i) holds the
 *             min(k_sel, pos-w+1) candidates with the highest group score
 *                 a[j] = max over the query heads h of group g of (scale*<q_h,k_j> - LSE_h)
 *             (the log of the largest softmax probability any head of the group gives key j),
 *             ties to the lower key index, written in ascending key order and padded with -1.
 *   scores_dbg out, NULL or float [batch, n_kv_heads, q_len, kv_len]: the a[j] the selection used
 *             (-inf for keys the query cannot see).  Meant for small problems and tests.
 *   ws   scratch for the score strips (unused when idx is NULL or scores_dbg is given).
 *             hs2_workspace_bytes(p, HS2_OP_FULL_ATTN_SELECT) is the recommended size (all rows, at most
 *             1 GiB); any 256-byte aligned buffer of at least 16*ceil(kv_len/4) bytes is accepted, a
 *             smaller one only means that fewer query rows are scored per launch.
 */
hs2_status hs2_full_attn_select(const hs2_problem *p, const void *Q, const void *K, const void *V,
                                void *O, float *LSE, int32_t *idx, float *scores_dbg,
                                void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Token-level top-k outside the window (Section 3.3) on caller-provided scores.
 *   scores in  float [batch, n_kv_heads, q_len, kv_len], packed.  Any finite floats or infinities;
 *              +0 and -0 compare equal; NaN is a caller error.
 *   idx    out as above.  The result is a pure function of the score bits: equal inputs give equal
 *              indices (order: score descending, then key index ascending).
 * head_dim, n_q_heads, dtype and the strides of `p` are ignored.
 */
hs2_status hs2_topk_select(const hs2_problem *p, const float *scores, int32_t *idx,
                           void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * SA layer, prefill (Section 3.3: the recent window is always part of the attended set, the k best-scoring
 * tokens outside it come from the FA layer's selection, and K/V of both are read from the FA layer's cache).
 *   Q     in  this SA layer's own queries; K, V: the FA layer's cache; idx: the FA layer's indices.
 *   An idx entry is ignored when it is negative, greater than pos-w (inside the window or in the
 *   future) or >= kv_lens[b]; the attended set is the union with the window and no entry can cause
 *   an out-of-bounds read.  Repeating an index inside one row is a caller error (it is counted twice).
 *   sink  in  NULL or float [n_q_heads]: per-head sink bias added to the softmax denominator only
 *             (Section 4.1: sparse layers use learnable per-head sink biases).
 *   O     out; LSE out, nullable.  A query whose attended set is empty gets O = 0, LSE = -inf.
 */
hs2_status hs2_sparse_attn_prefill(const hs2_problem *p, const void *Q, const void *K, const void *V,
                                   const int32_t *idx, const float *sink, void *O, float *LSE,
                                   void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * SA layer, decode: q_len must be 1 (one new token per sequence, its K/V already in the cache).
 * The attended set of each (sequence, KV head) is split over several warps; the partial results
 * are merged on the device by the last split to finish (no kernel waits on another).
 * Arguments as for the prefill call.
 */
hs2_status hs2_sparse_attn_decode(const hs2_problem *p, const void *Q, const void *K, const void *V,
                                  const int32_t *idx, const float *sink, void *O, float *LSE,
                                  void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The two SA calls with the sigmoid output gate of the sparse layers fused into the store (Section 4.1 gives the
 * sparse and the sliding-window layers such gates): O = sigmoid(gate) * attention output, elementwise.
 *   gate  in  the gate logits (the caller's projection of the layer input; not computed here): shape, dtype
 *             and strides of O (p->o_stride).  Must not be NULL (use the ungated call instead).
 * LSE is not affected by the gate.  Everything else as for the ungated calls.
 */
hs2_status hs2_sparse_attn_prefill_gated(const hs2_problem *p, const void *Q, const void *K, const void *V,
                                         const int32_t *idx, const float *sink, const void *gate, void *O,
                                         float *LSE, void *ws, size_t ws_bytes, void *cuda_stream);
hs2_status hs2_sparse_attn_decode_gated(const hs2_problem *p, const void *Q, const void *K, const void *V,
                                        const int32_t *idx, const float *sink, const void *gate, void *O,
                                        float *LSE, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The two SA calls on an FP8 KV cache (the storage format the paper's cost analysis of Section 4 assumes; the
 * paper gives no quantisation recipe, this is the usual one):
 *   K8, V8   in  e4m3 codes (1 byte: sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities, the two
 *                NaN codes are a caller error) [batch, kv_len, n_kv_heads, head_dim]; p->kv_stride counts codes
 *                (= bytes), multiples of 16, or 0 for packed.
 *   k_scale, v_scale  in  float [batch, kv_len, n_kv_heads]: the cache value is code * scale.  Packed, or with the
 *                strides p->kv_scale_stride gives (floats; shared by the two arrays).  Codes and scales may live in one
 *                buffer of records, e.g. 288 bytes [K codes | V codes | K scale | V scale | spare] per (token, KV head)
 *                at head_dim 128 (hs2_kv_project_fp8_records writes that): an attended token then costs a sparse
 *                layer one DRAM page instead of four (9 % off its decode step at 64K), while the full layer's sweep
 *                over the whole cache reads the spare bytes too (7 % more).
 *   Q, O, LSE, idx, sink as for the bf16 calls; p->dtype describes Q and O and must be HS2_BF16.
 * Covers head_dim 128 and 256 with up to 128 query heads per KV head (the paper's own shape, 64 heads on one KV
 * head at head_dim 256, included) and 16-byte aligned tensors; anything else returns HS2_ERR_UNSUPPORTED.  At
 * head_dim 128 with groups of up to 8 (or 16) heads the codes are converted on their way into the mma.sync
 * operands and V scales up to 255 are supported (probability x scale is carried in an f16 operand); every other
 * shape runs on the tcgen05 gather kernel, whose gather warps dequantise into bf16 operands.
 * No scratch is needed: decode runs one CTA per (sequence, KV head) on the mma.sync kernel; on the tcgen05 kernel
 * the CTAs that split a sequence's keys form a thread-block cluster and merge through distributed shared memory.
 */
hs2_status hs2_sparse_attn_prefill_fp8kv(const hs2_problem *p, const void *Q, const void *K8, const void *V8,
                                         const float *k_scale, const float *v_scale, const int32_t *idx,
                                         const float *sink, void *O, float *LSE, void *cuda_stream);
hs2_status hs2_sparse_attn_decode_fp8kv(const hs2_problem *p, const void *Q, const void *K8, const void *V8,
                                        const float *k_scale, const float *v_scale, const int32_t *idx,
                                        const float *sink, void *O, float *LSE, void *cuda_stream);

/*
 * The decode step of the full-attention layer on the FP8 cache (Section 3.4, with the cache storage that the cost
 * analysis of Section 4 assumes): one query per sequence attends to its whole context, and the layer selects the
 * k_sel tokens outside the window from the same scores, exactly as hs2_full_attn_select does on a bf16 cache.
 *   Q [B,1,Hq,D] bf16; K8, V8, k_scale, v_scale: the cache as described above for the sparse calls; O [B,1,Hq,D] bf16;
 *   LSE [B,Hq,1] fp32; idx [B,Hkv,1,k_sel] int32 or NULL (attention only).  All device pointers.
 *   ws: with idx, at least hs2_workspace_bytes(p, HS2_OP_FULL_ATTN_SELECT_FP8KV) bytes, 256-byte aligned (the
 *   dequantised q.k products of every head and key, 4 bytes each, and one score row per (sequence, KV head));
 *   HS2_ERR_WORKSPACE_TOO_SMALL otherwise.  Without idx no scratch is needed.
 *   Covers q_len == 1, 16-byte aligned tensors, head_dim 128 or 256 with up to 128 query heads per KV head (at
 *   head_dim 128 and groups of at most 8 the cache is swept once and the products kept, which must fit 2 GiB; other
 *   shapes sweep K a second time for the scores); anything else returns HS2_ERR_UNSUPPORTED and launches nothing.
 *   (A prefill-shaped full layer attends to the bf16 K and V it has just produced, so there is no FP8 variant of it.)
 */
hs2_status hs2_full_attn_select_fp8kv(const hs2_problem *p, const void *Q, const void *K8, const void *V8,
                                      const float *k_scale, const float *v_scale, void *O, float *LSE, int32_t *idx,
                                      void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * hs2_sparse_attn_decode for callers that cannot hand over a scratch buffer.  (The paper has no
 * counterpart to this call; it is a packaging variant of the decode operator above.)
 *
 * Who needs it: code that is not allowed to obtain device memory at the point where it decodes -
 * a plugin that is given nothing but the tensors' pointers, a server that handed the whole device
 * to its own pool at start-up and has none left to carve a workspace from, a latency-critical loop
 * that cannot afford the device-wide synchronisation an allocation implies.  For them the partial
 * results of the split kernel live in an array that is part of the library image:
 * 8,519,936 bytes on every GPU that loads the library, held until the process exits.
 *
 *   - Same arguments and results as hs2_sparse_attn_decode, minus `ws`.  The call allocates nothing
 *     and frees nothing, on the host or on the device.
 *   - Limit: at most HS2_STATIC_DECODE_MAX_PAIRS (64) units of work, a unit being one (sequence,
 *     KV head) with up to 8 query heads: batch * n_kv_heads <= 64 for groups of up to 8 heads; a
 *     group of 16 heads runs as two units, so batch * n_kv_heads <= 32 there.  A larger problem
 *     returns HS2_ERR_STATIC_SCRATCH and launches nothing.  It covers what the tensor-core decode
 *     kernel covers (bf16, head_dim 128, groups of up to 8 or of 16 heads, 16-byte aligned tensors);
 *     anything else returns HS2_ERR_UNSUPPORTED.
 *   - The first call on each device looks up the array's device address; make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one array, which still holds the previous call's data: the
 *     call clears the part that must start at zero itself, and two calls whose kernels can overlap
 *     on the GPU (different streams, no ordering between them) race on it.  Order them.
 */
#define HS2_STATIC_DECODE_MAX_PAIRS 64
hs2_status hs2_sparse_attn_decode_static(const hs2_problem *p, const void *Q, const void *K, const void *V,
                                         const int32_t *idx, const float *sink, void *O, float *LSE,
                                         void *cuda_stream);

/*
 * Producer of the caches the calls above read (Section 3.2, KV Bridging: K_j = Proj^K_j(H_i), V_j = Proj^V_j(H_i);
 * several layers fed from one hidden-state source are simply more output columns):  C = H W^T.
 *   H       in  bf16 [n_tokens, d_model], row stride ldh (elements)
 *   W       in  bf16 [n_out, d_model], row stride ldw: one row per output feature (a linear layer's weight)
 *   C       out [n_tokens, n_out] with row stride ldc, so that it can be a cache [.., tokens, n_kv_heads, head_dim]
 *               or a slice of a fused one.  scales == NULL: bf16 (ldc in elements).  scales != NULL: e4m3 codes
 *               (ldc in bytes) and
 *   scales  out float [n_tokens, n_out / 128], packed: one scale per token and group of 128 consecutive columns
 *               (= one head of dim 128): amax / 448 (1 for an all-zero group); code = value / scale rounded to
 *               nearest even.  This is the format hs2_sparse_attn_*_fp8kv reads.
 * d_model % 64 == 0, n_out % 256 == 0, strides multiples of 8 elements (16 bytes for the e4m3 output), 16-byte
 * aligned pointers; anything else returns HS2_ERR_UNSUPPORTED.  fp32 accumulation; no scratch.
 */
hs2_status hs2_kv_project(int64_t n_tokens, int32_t d_model, int32_t n_out, const void *H, int64_t ldh, const void *W,
                          int64_t ldw, void *C, int64_t ldc, float *scales, void *cuda_stream);

/*
 * The e4m3 form of hs2_kv_project writing into a cache of records, so that the K codes, the V codes and both scales
 * of a (token, KV head) can sit side by side (one DRAM page per attended token and head instead of four; on the 64K
 * decode step of the benchmark a sparse layer then takes 39.7 us instead of 43.7, the full layer 1.13 ms instead of 1.04).  A column group g is the 128
 * consecutive output columns 128 g .. 128 g + 127 (one head of dim 128):
 *   codes of token t, group g   at byte  t * ldc + g * ld_group  of C   (128 bytes)
 *   their scale                 at       scales[t * scale_ld_token + g * scale_ld_group]
 * Example, records of 288 bytes [K 128 | V 128 | K scale | V scale | 24 spare] per (token, KV head) - a whole number
 * of 32-byte sectors, which measured 39.7 us against 40.7 us for records of 272 bytes - with n_kv_heads heads: the K
 * projection is called with C = cache, ldc = 288 n_kv_heads, ld_group = 288, scales = (float *)(cache + 256),
 * scale_ld_token = 72 n_kv_heads, scale_ld_group = 72; the V projection with C = cache + 128 and
 * scales = (float *)(cache + 260).  The attention calls read such a cache through kv_stride = {tokens * 288 n_kv_heads,
 * 288 n_kv_heads, 288} and kv_scale_stride = {tokens * 72 n_kv_heads, 72 n_kv_heads, 72}.
 * ld_group >= 128; ldc and ld_group multiples of 16 bytes; ldc >= (n_out / 128 - 1) * ld_group + 128; the other
 * conditions and the arithmetic are those of hs2_kv_project.
 */
hs2_status hs2_kv_project_fp8_records(int64_t n_tokens, int32_t d_model, int32_t n_out, const void *H, int64_t ldh,
                                      const void *W, int64_t ldw, void *C, int64_t ldc, int64_t ld_group, float *scales,
                                      int64_t scale_ld_token, int64_t scale_ld_group, void *cuda_stream);

/*
 * Measurement aid for hs2_sparse_attn_prefill (the gather of Section 3.3; no counterpart in the paper): performs
 * only the row fetches of that call - the same work items in the same order, the same slot array [idx row | forced
 * window] with the same validity rules, every attended K row and V row loaded with 16-byte loads - and no
 * arithmetic.  Its duration is what the memory system needs to deliver the rows to the SMs: the ceiling for the
 * attention call's gather on this problem, whether the cache sits in L2 or in HBM.
 *   p, K, V, idx  as for hs2_sparse_attn_prefill (bf16, head_dim 128, 16-byte aligned K and V; else
 *                 HS2_ERR_UNSUPPORTED).  Q and O are not touched.
 *   mode          0: loads that bypass L1 (what the attention kernel's copies do); 1: loads through L1.
 *   sink_word     device, one unsigned the caller zeroes; it only keeps the loads observable.
 */
hs2_status hs2_probe_gather(const hs2_problem *p, const void *K, const void *V, const int32_t *idx, int mode,
                            unsigned *sink_word, void *cuda_stream);

/* Static, never-NULL description of a status. */
const char *hs2_status_string(hs2_status s);

/* The cudaError_t (as int) behind the calling thread's most recent HS2_ERR_CUDA, 0 if none. */
int hs2_last_cuda_error(void);

/* Reads the library's device error word into *flags (0 = fine).  One byte per kernel family:
 *   bits  0-7   full-attention and score-sweep kernels (tcgen05)
 *   bits  8-15  sparse-attention kernels on mma.sync (bf16 and FP8 cache)
 *   bits 16-23  sparse-attention kernel on tcgen05
 *   bits 24-31  KV projection
 * Within a byte, bit 0: a bounded wait inside a kernel ran out and that kernel abandoned its work (its
 * output is then incomplete); bit 1: a kernel refused a misaligned shared-memory window.  Test
 * `flags != 0`, not single bits.  Sticky until the process exits.  Synchronises the current device.
 * Returns an hs2_status. */
int hs2_device_error_flags(unsigned *flags);

/* Testing knob: enabled = 0 makes hs2_full_attn_select use its mma.sync kernels (the path taken when TMA
 * tensor maps cannot be built) instead of the tcgen05 ones; 1 restores the default; negative only queries.
 * Returns the previous setting.  Process-wide. */
int hs2_set_tcgen05_enabled(int enabled);

/* Tuning knob of hs2_full_attn_select: from which kv_len on (default 18432) the selection thresholds a sample of
 * the scores and works on filtered candidate lists instead of complete score strips.  Both ways select from the same
 * tensor-core scores and give the same indices, with one exception: a row whose filtered list came out unusable
 * is redone from scores recomputed with fp32 FMAs, which can order two keys differently when their scores agree
 * to within rounding (inside the 1e-3 near-tie band).  Returns the previous value; min_keys <= 0 only queries.
 * Process-wide, read at the start of each call: set it before calls start on other threads. */
int hs2_set_filter_min_keys(int min_keys);

/* Number of kernels this library has launched in the process so far (all threads, all streams). */
unsigned long long hs2_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* HS2_H_ */
