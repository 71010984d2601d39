// Measurement aid for the sparse layers (Section 3.3): the row fetches of the sparse-attention prefill, and nothing
// else.  The kernel walks the same work items in the same order as the attention kernel - one warp per (sequence,
// KV head, query), queries fastest - resolves the same slot array [index row | forced window] with the same validity
// rules, and loads every attended K row and V row (head_dim 128 bf16 = 256 bytes each) with 16-byte loads, sixteen
// lanes per row.  The loaded words are folded with XOR into one value per warp, so that the loads cannot be removed.
// No shared memory, no tensor cores, full occupancy: its duration is what the memory system (L2 when the cache of a
// KV head is resident there, HBM otherwise) needs to deliver those rows to the SMs, i.e. the ceiling that the
// attention kernel's gather can approach but not beat.
#include "hs2_common.cuh"

namespace hs2 {
namespace {

template <bool L1>
__device__ __forceinline__ uint4 load16(const char *p)
{
    uint4 v;
    if (L1)
        asm volatile("ld.global.nc.L1::evict_last.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    else
        asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

constexpr int kProbeWarps = 8;

template <bool L1>
__global__ void __launch_bounds__(kProbeWarps * 32)
k_probe_gather(const Params p, const __nv_bfloat16 *__restrict__ K, const __nv_bfloat16 *__restrict__ V,
               const int32_t *__restrict__ idx, unsigned *__restrict__ out)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t item = (int64_t)blockIdx.x * kProbeWarps + warp;   // (b, g, i), i fastest
    if (item >= (int64_t)p.B * p.Hkv * p.Lq) return;
    const int i = (int)(item % p.Lq);
    const int g = (int)((item / p.Lq) % p.Hkv);
    const int b = (int)(item / ((int64_t)p.Lq * p.Hkv));
    const int pos = pos_of(p, b, i), kvl = kvlen_of(p, b);
    const int64_t base = b * p.ks_b + g * p.ks_h;
    const int c = lane & 15, hi = lane >> 4;
    const char *kc = reinterpret_cast<const char *>(K + base) + c * 16;
    const char *vc = reinterpret_cast<const char *>(V + base) + c * 16;
    const int64_t rs = p.ks_t * 2;
    const int32_t *irow = idx ? idx + (((int64_t)b * p.Hkv + g) * p.Lq + i) * p.k : nullptr;
    const int n_slots = p.k + p.w;
    uint4 acc = make_uint4(0u, 0u, 0u, 0u);
    for (int s0 = 0; s0 < n_slots; s0 += 32) {
        const int s = s0 + lane;
        int j = -1;
        if (s < p.k) j = irow ? __ldg(irow + s) : -1;
        else if (s < n_slots) j = pos - p.w + 1 + (s - p.k);
        const int top = s < p.k ? pos - p.w : pos;   // index entries inside the window are void
        if (j < 0 || j > top || j >= kvl) j = -1;
        if (!__ballot_sync(0xffffffffu, j >= 0)) continue;
#pragma unroll
        for (int r0 = 0; r0 < 32; r0 += 8) {
            uint4 kv[4], vv[4];
            int jr[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                jr[u] = __shfl_sync(0xffffffffu, j, r0 + 2 * u + hi);
                const int64_t off = (int64_t)max(jr[u], 0) * rs;
                if (jr[u] >= 0) {
                    kv[u] = load16<L1>(kc + off);
                    vv[u] = load16<L1>(vc + off);
                } else {
                    kv[u] = vv[u] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                acc.x ^= kv[u].x ^ vv[u].x; acc.y ^= kv[u].y ^ vv[u].y;
                acc.z ^= kv[u].z ^ vv[u].z; acc.w ^= kv[u].w ^ vv[u].w;
            }
        }
    }
    unsigned r = acc.x ^ acc.y ^ acc.z ^ acc.w;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) r ^= __shfl_xor_sync(0xffffffffu, r, o);
    if (lane == 0 && r == 0x9e3779b9u) atomicAdd(out, 1u);   // practically never true; keeps the loads alive
}

}  // namespace

cudaError_t launch_probe_gather(const Params &p, const void *K, const void *V, const int32_t *idx, int mode,
                                unsigned *out, cudaStream_t st)
{
    const int64_t items = (int64_t)p.B * p.Hkv * p.Lq;
    const int64_t blocks = (items + kProbeWarps - 1) / kProbeWarps;
    if (blocks <= 0 || blocks > 0x7fffffff) return cudaErrorNotSupported;
    auto *k = static_cast<const __nv_bfloat16 *>(K);
    auto *v = static_cast<const __nv_bfloat16 *>(V);
    if (mode == 1) k_probe_gather<true><<<(unsigned)blocks, kProbeWarps * 32, 0, st>>>(p, k, v, idx, out);
    else k_probe_gather<false><<<(unsigned)blocks, kProbeWarps * 32, 0, st>>>(p, k, v, idx, out);
    count_launch();
    return cudaGetLastError();
}

}  // namespace hs2
