// Full-attention layer on tensor cores (bf16, head_dim 128): causal flash-style attention that
// produces O and LSE, and the score sweep that turns the layer's exact attention scores into the
// per-(query, KV head) selection scores a[j] = max_h (scale <q_h, k_j> - LSE_h)   (Section 3.4).
//
// k_full_mma   : one CTA = 128 queries of one head, 8 warps x 16 rows, K/V tiles of 64 keys double
//                buffered with cp.async, S = Q K^T and O += P V with mma.sync m16n8k16, online softmax
//                in the base-2 domain.  Diagonal tiles are masked per element, tiles above a warp's
//                rows are skipped.
// k_scores_mma : one warp = 8 queries x all G heads of a group; keys ride on the MMA M dimension and
//                the 8 queries on N, so one K fragment feeds all G heads.  -LSE_h/scale enters as the
//                accumulator's initial value, so each head costs 8 MMAs and 4 max operations per
//                16 keys x 8 queries.  Results are staged in shared memory and written as full rows.
#include "hs2_common.cuh"

namespace hs2 {
namespace {

constexpr int HD = 128;
constexpr int kRowBytes = HD * 2;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16_c(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1, const float (&c)[4])
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};\n"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// rows of 256 bytes, 16-byte chunk c of row r stored at chunk position c ^ (r & 7)
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return row * kRowBytes + ((chunk ^ (row & 7)) << 4); }

// Copy `rows` rows (256 B each) of a token-major tensor into a swizzled tile; rows at or beyond
// `limit` (and before 0) are zero filled.
__device__ __forceinline__ void load_tile(uint32_t sdst, const char *gbase, int64_t row_stride_bytes, int first_row,
                                          int rows, int limit, int tid, int nthreads)
{
    for (int e = tid; e < rows * 16; e += nthreads) {
        const int r = e >> 4, c = e & 15;
        const int gr = first_row + r;
        const bool ok = gr >= 0 && gr < limit;
        cp_async16(sdst + swz(r, c), gbase + (int64_t)(ok ? gr : 0) * row_stride_bytes + c * 16, ok ? 16 : 0);
    }
}

// ---------------------------------------------------------------- causal attention, O and LSE
constexpr int BM = 128, BN = 64, FA_WARPS = 8;
constexpr int kFaSmem = BM * kRowBytes + 2 * 2 * BN * kRowBytes;   // Q tile + double-buffered K and V tiles

__global__ void __launch_bounds__(FA_WARPS * 32, 1)
k_full_mma(const Params p, const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
           const __nv_bfloat16 *__restrict__ V, __nv_bfloat16 *__restrict__ O, float *__restrict__ LSE)
{
    extern __shared__ __align__(128) char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3, mi = lane >> 3, rr = lane & 7;
    const int mblk = gridDim.x - 1 - blockIdx.x;   // long rows first
    const int h = blockIdx.y % p.Hq, b = blockIdx.y / p.Hq;
    const int gkv = h / p.G;
    const int i0 = mblk * BM;
    const int kvl = kvlen_of(p, b);
    const int pos0 = pos_of(p, b, i0);
    const int rows_here = min(BM, p.Lq - i0);
    const int n_vis = max(0, min(pos0 + rows_here, kvl));   // keys any row of the tile can see
    const int nblk = (n_vis + BN - 1) / BN;

    const uint32_t sQ = smem_u32(smem);
    const uint32_t sK = sQ + BM * kRowBytes;
    const uint32_t sV = sK + 2 * BN * kRowBytes;
    const char *qb = reinterpret_cast<const char *>(Q + b * p.qs_b + h * p.qs_h);
    const char *kb = reinterpret_cast<const char *>(K + b * p.ks_b + gkv * p.ks_h);
    const char *vb = reinterpret_cast<const char *>(V + b * p.ks_b + gkv * p.ks_h);
    const int64_t qrs = p.qs_t * 2, krs = p.ks_t * 2;

    load_tile(sQ, qb, qrs, i0, BM, p.Lq, tid, FA_WARPS * 32);
    if (nblk > 0) {
        load_tile(sK, kb, krs, 0, BN, kvl, tid, FA_WARPS * 32);
        load_tile(sV, vb, krs, 0, BN, kvl, tid, FA_WARPS * 32);
    }
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();

    uint32_t qf[8][4];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) ldmatrix_x4(qf[ks], sQ + swz(warp * 16 + (mi & 1) * 8 + rr, 2 * ks + (mi >> 1)));

    float o[16][4];
#pragma unroll
    for (int dn = 0; dn < 16; ++dn) o[dn][0] = o[dn][1] = o[dn][2] = o[dn][3] = 0.f;
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    const int prow[2] = {pos0 + warp * 16 + g, pos0 + warp * 16 + g + 8};   // absolute position of this thread's rows
    const int warp_last = pos0 + warp * 16 + 15;

    for (int jb = 0; jb < nblk; ++jb) {
        const int st = jb & 1;
        if (jb + 1 < nblk) {
            load_tile(sK + (st ^ 1) * BN * kRowBytes, kb, krs, (jb + 1) * BN, BN, kvl, tid, FA_WARPS * 32);
            load_tile(sV + (st ^ 1) * BN * kRowBytes, vb, krs, (jb + 1) * BN, BN, kvl, tid, FA_WARPS * 32);
        }
        cp_async_commit();
        if (jb > 0) {
            cp_async_wait<1>();
            __syncthreads();
        }
        const int j0 = jb * BN;
        if (j0 <= warp_last) {   // otherwise every key of the tile is in this warp's future
            const uint32_t kt = sK + st * BN * kRowBytes, vt = sV + st * BN * kRowBytes;
            float s[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    uint32_t kf[4];
                    ldmatrix_x4(kf, kt + swz(np * 16 + (mi >> 1) * 8 + rr, 2 * ks + (mi & 1)));
                    mma_bf16(s[2 * np], qf[ks], kf[0], kf[1]);
                    mma_bf16(s[2 * np + 1], qf[ks], kf[2], kf[3]);
                }
            }
            const bool need_mask = (j0 + BN - 1 > pos0 + warp * 16) || (j0 + BN > kvl);
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = s[nt][e] * p.scale_log2;
                    if (need_mask) {
                        const int j = j0 + nt * 8 + 2 * t + (e & 1);
                        if (j > prow[e >> 1] || j >= kvl) v = -INFINITY;
                    }
                    s[nt][e] = v;
                    mx[e >> 1] = fmaxf(mx[e >> 1], v);
                }
            float corr[2], muse[2];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
                mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
                const float m_new = fmaxf(m[r], mx[r]);
                muse[r] = m_new == -INFINITY ? 0.f : m_new;
                corr[r] = exp2f(m[r] - muse[r]);
                m[r] = m_new;
                l[r] *= corr[r];
            }
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float pv = exp2f(s[nt][e] - muse[e >> 1]);
                    s[nt][e] = pv;
                    l[e >> 1] += pv;
                }
#pragma unroll
            for (int dn = 0; dn < 16; ++dn) {
                o[dn][0] *= corr[0]; o[dn][1] *= corr[0];
                o[dn][2] *= corr[1]; o[dn][3] *= corr[1];
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {   // 16 keys per step
                uint32_t pa[4];
                pa[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
                pa[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
                pa[2] = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
                pa[3] = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
                for (int dp = 0; dp < 8; ++dp) {
                    uint32_t vf[4];
                    ldmatrix_x4_trans(vf, vt + swz(kk * 16 + (mi & 1) * 8 + rr, 2 * dp + (mi >> 1)));
                    mma_bf16(o[2 * dp], pa, vf[0], vf[1]);
                    mma_bf16(o[2 * dp + 1], pa, vf[2], vf[3]);
                }
            }
        }
        __syncthreads();   // the stage is free for the load issued two iterations later
    }
    cp_async_wait<0>();

    // epilogue: normalise, stage the warp's 16 rows in the (no longer needed) Q tile, store full rows
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l[r] += __shfl_xor_sync(0xffffffffu, l[r], 1);
        l[r] += __shfl_xor_sync(0xffffffffu, l[r], 2);
    }
    const float inv[2] = {l[0] > 0.f ? 1.f / l[0] : 0.f, l[1] > 0.f ? 1.f / l[1] : 0.f};
    char *stage = smem;   // rows warp*16 .. +15 of the Q tile belong to this warp alone
#pragma unroll
    for (int dn = 0; dn < 16; ++dn)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int row = warp * 16 + g + 8 * r;
            const uint32_t off = swz(row, dn) + t * 4;
            *reinterpret_cast<uint32_t *>(stage + off) = pack_bf16(o[dn][2 * r] * inv[r], o[dn][2 * r + 1] * inv[r]);
        }
    __syncwarp();
    for (int e = lane; e < 16 * 16; e += 32) {
        const int r = warp * 16 + (e >> 4), c = e & 15;
        const int i = i0 + r;
        if (i < p.Lq) {
            const uint4 val = *reinterpret_cast<const uint4 *>(stage + swz(r, c));
            *reinterpret_cast<uint4 *>(O + b * p.os_b + i * p.os_t + h * p.os_h + c * 8) = val;
        }
    }
    if (t == 0) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int i = i0 + warp * 16 + g + 8 * r;
            if (i < p.Lq)
                LSE[((int64_t)b * p.Hq + h) * p.Lq + i] = l[r] > 0.f ? (m[r] + log2f(l[r])) * kLn2 : -INFINITY;
        }
    }
}

// ---------------------------------------------------------------- group selection scores
constexpr int SC_WARPS = 8, SC_Q = 8 * SC_WARPS, SC_KT = 64, SC_CHUNK = 2048;
constexpr int kScSmem = 2 * SC_KT * kRowBytes + SC_WARPS * 8 * SC_KT * 4;   // K double buffer + per-warp staging

template <int G>
__global__ void __launch_bounds__(SC_WARPS * 32, 1)
k_scores_mma(const Params p, const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
             const float *__restrict__ LSE, float *__restrict__ out, int64_t out_stride, int64_t row0, int64_t n_rows,
             int all_visible, int tile_first, int tiles_per_bg, int vec_ok)
{
    extern __shared__ __align__(128) char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3, mi = lane >> 3, rr = lane & 7;
    const int tile = tile_first + blockIdx.y;   // flattened (b, g, query tile)
    const int bg = tile / tiles_per_bg;
    const int qt = tile % tiles_per_bg;
    const int gkv = bg % p.Hkv, b = bg / p.Hkv;
    const int kvl = kvlen_of(p, b);
    const int iq0 = qt * SC_Q;                                // first query of the CTA
    // rows of this (b, g) that belong to the requested block
    const int64_t bg_row0 = (int64_t)bg * p.Lq;
    const int i_lo = (int)max((int64_t)0, row0 - bg_row0), i_hi = (int)min((int64_t)p.Lq, row0 + n_rows - bg_row0);
    const int c_lo = max(iq0, i_lo), c_hi = min(iq0 + SC_Q, i_hi);   // queries this CTA really owns
    if (c_lo >= c_hi) return;
    auto n_of = [&](int i) {   // how many leading keys row i needs
        const int pos = pos_of(p, b, i);
        return max(0, min(all_visible ? pos + 1 : pos - p.w + 1, kvl));
    };
    const int limit = n_of(c_hi - 1);
    const int key0 = blockIdx.x * SC_CHUNK;
    const int key_end = min(limit, key0 + SC_CHUNK);
    if (key0 >= key_end) return;

    const uint32_t sK = smem_u32(smem);
    float *stage = reinterpret_cast<float *>(smem + 2 * SC_KT * kRowBytes) + warp * 8 * SC_KT;
    const char *kb = reinterpret_cast<const char *>(K + b * p.ks_b + gkv * p.ks_h);
    const int64_t krs = p.ks_t * 2;

    // this warp's 8 queries
    const int wq0 = iq0 + warp * 8;
    const int my_i = wq0 + g;                                 // the query whose Q fragment this thread holds
    const bool my_ok = my_i >= c_lo && my_i < c_hi;
    uint32_t qf[G][16];
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
        if (my_ok) {
            const uint32_t *q = reinterpret_cast<const uint32_t *>(Q + b * p.qs_b + (int64_t)my_i * p.qs_t + (gkv * G + hh) * p.qs_h);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) { qf[hh][2 * ks] = __ldg(q + ks * 8 + t); qf[hh][2 * ks + 1] = __ldg(q + ks * 8 + 4 + t); }
        } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) qf[hh][e] = 0u;
        }
    }
    // -LSE/scale of the two queries whose columns this thread accumulates (queries 2t, 2t+1 of the warp)
    const float inv_scale = 1.f / p.scale;
    float nl[G][2];
    int n_row[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int i = wq0 + 2 * t + e;
        const bool ok = i >= c_lo && i < c_hi;
        n_row[e] = ok ? n_of(i) : 0;
#pragma unroll
        for (int hh = 0; hh < G; ++hh)
            nl[hh][e] = ok ? -LSE[((int64_t)b * p.Hq + gkv * G + hh) * p.Lq + i] * inv_scale : 0.f;
    }
    int warp_n = 0;   // keys needed by any query of this warp
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const int i = wq0 + e;
        if (i >= c_lo && i < c_hi) warp_n = max(warp_n, n_of(i));
    }

    const int ntile = (key_end - key0 + SC_KT - 1) / SC_KT;
    load_tile(sK, kb, krs, key0, SC_KT, kvl, tid, SC_WARPS * 32);
    cp_async_commit();
    for (int tt = 0; tt < ntile; ++tt) {
        const int st = tt & 1;
        if (tt + 1 < ntile) load_tile(sK + (st ^ 1) * SC_KT * kRowBytes, kb, krs, key0 + (tt + 1) * SC_KT, SC_KT, kvl, tid, SC_WARPS * 32);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const int j0 = key0 + tt * SC_KT;
        if (j0 < warp_n) {
            const uint32_t kt = sK + st * SC_KT * kRowBytes;
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) {
                uint32_t a[8][4];
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) ldmatrix_x4(a[ks], kt + swz(mt * 16 + (mi & 1) * 8 + rr, 2 * ks + (mi >> 1)));
                float amax[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int hh = 0; hh < G; hh += 2) {
                    float acc0[4], acc1[4];
                    const float c0[4] = {nl[hh][0], nl[hh][1], nl[hh][0], nl[hh][1]};
                    mma_bf16_c(acc0, a[0], qf[hh][0], qf[hh][1], c0);
                    if (hh + 1 < G) {
                        const float c1[4] = {nl[hh + 1 < G ? hh + 1 : hh][0], nl[hh + 1 < G ? hh + 1 : hh][1],
                                             nl[hh + 1 < G ? hh + 1 : hh][0], nl[hh + 1 < G ? hh + 1 : hh][1]};
                        mma_bf16_c(acc1, a[0], qf[hh + 1 < G ? hh + 1 : hh][0], qf[hh + 1 < G ? hh + 1 : hh][1], c1);
                    }
#pragma unroll
                    for (int ks = 1; ks < 8; ++ks) {
                        mma_bf16(acc0, a[ks], qf[hh][2 * ks], qf[hh][2 * ks + 1]);
                        if (hh + 1 < G) mma_bf16(acc1, a[ks], qf[hh + 1 < G ? hh + 1 : hh][2 * ks], qf[hh + 1 < G ? hh + 1 : hh][2 * ks + 1]);
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        amax[e] = fmaxf(amax[e], acc0[e]);
                        if (hh + 1 < G) amax[e] = fmaxf(amax[e], acc1[e]);
                    }
                }
                // thread holds (key g, query 2t), (key g, query 2t+1), (key g+8, query 2t), (key g+8, query 2t+1)
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    stage[(2 * t + (e & 1)) * SC_KT + mt * 16 + g + 8 * (e >> 1)] = amax[e] * p.scale;
            }
            __syncwarp();
            // write the 8 rows of 64 keys: 16 lanes x float4 per row
            const int c4 = (lane & 15) * 4;
#pragma unroll
            for (int qq = 0; qq < 8; qq += 2) {
                const int q = qq + (lane >> 4);
                const int i = wq0 + q;
                if (i >= c_lo && i < c_hi) {
                    const int n = n_of(i);
                    float *orow = out + (bg_row0 + i - row0) * out_stride;
                    const int j = j0 + c4;
                    const float4 v = *reinterpret_cast<const float4 *>(stage + q * SC_KT + c4);
                    if (vec_ok && j + 4 <= n) {
                        *reinterpret_cast<float4 *>(orow + j) = v;
                    } else {
                        if (j < n) orow[j] = v.x;
                        if (j + 1 < n) orow[j + 1] = v.y;
                        if (j + 2 < n) orow[j + 2] = v.z;
                        if (j + 3 < n) orow[j + 3] = v.w;
                    }
                }
            }
            __syncwarp();
        }
        __syncthreads();
    }
    cp_async_wait<0>();
    (void)n_row;
}

__global__ void k_fill(float *__restrict__ out, int64_t n, float v)
{
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) out[e] = v;
}

bool g_attr_set[64] = {};
template <int G> cudaError_t set_score_attr()
{
    return cudaFuncSetAttribute(k_scores_mma<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, kScSmem);
}
cudaError_t set_attrs()
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && g_attr_set[dev]) return cudaSuccess;
    if ((e = cudaFuncSetAttribute(k_full_mma, cudaFuncAttributeMaxDynamicSharedMemorySize, kFaSmem)) != cudaSuccess) return e;
    if ((e = set_score_attr<1>()) != cudaSuccess) return e;
    if ((e = set_score_attr<2>()) != cudaSuccess) return e;
    if ((e = set_score_attr<4>()) != cudaSuccess) return e;
    if ((e = set_score_attr<8>()) != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) g_attr_set[dev] = true;
    return cudaSuccess;
}

}  // namespace

bool full_mma_supported(const Params &p, hs2_dtype dt)
{
    auto m8 = [](int64_t x) { return x % 8 == 0; };
    const bool g_ok = p.G == 1 || p.G == 2 || p.G == 4 || p.G == 8;
    return dt == HS2_BF16 && p.D == HD && g_ok && m8(p.qs_b) && m8(p.qs_t) && m8(p.qs_h) && m8(p.ks_b) && m8(p.ks_t) &&
           m8(p.ks_h) && m8(p.os_b) && m8(p.os_t) && m8(p.os_h) && (int64_t)p.B * p.Hq <= 65535;
}

cudaError_t launch_full_attn_mma(const Params &p, const void *Q, const void *K, const void *V, void *O, float *LSE,
                                 cudaStream_t st)
{
    cudaError_t e = set_attrs();
    if (e != cudaSuccess) return e;
    dim3 grid((p.Lq + BM - 1) / BM, p.B * p.Hq);
    k_full_mma<<<grid, FA_WARPS * 32, kFaSmem, st>>>(p, (const __nv_bfloat16 *)Q, (const __nv_bfloat16 *)K,
                                                     (const __nv_bfloat16 *)V, (__nv_bfloat16 *)O, LSE);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_scores_mma(const Params &p, const void *Q, const void *K, const float *LSE, float *out,
                              int64_t out_stride, int64_t row0, int64_t n_rows, bool all_visible, cudaStream_t st)
{
    if (n_rows == 0) return cudaSuccess;
    cudaError_t e = set_attrs();
    if (e != cudaSuccess) return e;
    if (all_visible) {   // keys a query cannot see read -inf
        const int64_t n = n_rows * out_stride;
        const int64_t fb = (n + 255) / 256;
        k_fill<<<(unsigned)(fb < 148 * 16 ? fb : 148 * 16), 256, 0, st>>>(out, n, -INFINITY);
        count_launch();
    }
    const int tiles_per_bg = (p.Lq + SC_Q - 1) / SC_Q;
    const int64_t last = row0 + n_rows - 1;
    const int64_t t_first = (row0 / p.Lq) * tiles_per_bg + (row0 % p.Lq) / SC_Q;
    const int64_t t_last = (last / p.Lq) * tiles_per_bg + (last % p.Lq) / SC_Q;
    const int64_t gy = t_last - t_first + 1;
    if (gy > 65535 || t_last > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const int bg_first = (int)t_first;
    dim3 grid((p.Lk + SC_CHUNK - 1) / SC_CHUNK, (unsigned)gy);
    const int vec_ok = (out_stride % 4 == 0) && (reinterpret_cast<uintptr_t>(out) % 16 == 0);
    const __nv_bfloat16 *q = (const __nv_bfloat16 *)Q, *k = (const __nv_bfloat16 *)K;
    switch (p.G) {
        case 1: k_scores_mma<1><<<grid, SC_WARPS * 32, kScSmem, st>>>(p, q, k, LSE, out, out_stride, row0, n_rows, all_visible, bg_first, tiles_per_bg, vec_ok); break;
        case 2: k_scores_mma<2><<<grid, SC_WARPS * 32, kScSmem, st>>>(p, q, k, LSE, out, out_stride, row0, n_rows, all_visible, bg_first, tiles_per_bg, vec_ok); break;
        case 4: k_scores_mma<4><<<grid, SC_WARPS * 32, kScSmem, st>>>(p, q, k, LSE, out, out_stride, row0, n_rows, all_visible, bg_first, tiles_per_bg, vec_ok); break;
        case 8: k_scores_mma<8><<<grid, SC_WARPS * 32, kScSmem, st>>>(p, q, k, LSE, out, out_stride, row0, n_rows, all_visible, bg_first, tiles_per_bg, vec_ok); break;
        default: return cudaErrorInvalidValue;
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace hs2
