"""Seeded synthetic inputs for the hybrid sparse-attention path.

This module only *draws inputs*: it holds none of the method's arithmetic
(no attention, no softmax, no selection).  The CPU oracle and the CUDA
path are both fed the bytes produced here, so neither depends on the other.

Every value is a pure function of ``(seed, tensor_id, flat_index)``:
a splitmix64 counter hash gives two 53-bit uniforms, Box-Muller (cosine
branch, fp64) turns them into one standard normal, which is then rounded
to fp32 / bf16.  Because the function is counter based, a tensor can be
produced in chunks, on the CPU or on a CUDA device, without keeping any
generator state.  A test always hands the *same* produced bytes to both
sides, so CPU/GPU libm differences in the last fp64 bit do not matter.

The workloads stand in for the attention layers of the paper's 80B-A3B
model on long agentic contexts (Section 4.1): shapes, budgets
(k global + w forced local tokens) and score structure (planted needles,
clustered keys) follow the benchmark configurations, not any dataset.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional

import torch

BASE_SEED = 260926368

# tensor ids (part of the hash counter)
TID_Q_FULL = 0
TID_K = 1
TID_V = 2
TID_Q_SPARSE0 = 10      # + layer index
TID_NEEDLE_POS = 100
TID_NEEDLE_TGT = 101
TID_NEEDLE_HEAD = 102
TID_CENTRES = 103
TID_CLUSTER_ID = 104

_M64 = (1 << 64) - 1


def _to_i64(x: int) -> int:
    """Python int (mod 2^64) -> signed 64-bit value torch can hold."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLD = _to_i64(0x9E3779B97F4A7C15)
_MUL1 = _to_i64(0xBF58476D1CE4E5B9)
_MUL2 = _to_i64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor holding uint64 bit patterns."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on int64 tensors (wrap-around arithmetic)."""
    z = z + _GOLD
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def _mix_int(z: int) -> int:
    z = (z + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def _stream_base(seed: int, tensor_id: int) -> int:
    """One 64-bit stream key per (seed, tensor)."""
    return _mix_int(_mix_int(seed) ^ ((tensor_id * 0xD1342543DE82EF95) & _M64))


def hash_u64(seed: int, tensor_id: int, index: torch.Tensor, lane: int = 0) -> torch.Tensor:
    """Counter hash: int64 tensor of uint64 bit patterns for each flat index."""
    base = _to_i64(_stream_base(seed, tensor_id))
    return _mix(index.to(torch.int64) * 2 + (base + lane))


def uniform_int(seed: int, tensor_id: int, index: torch.Tensor, n) -> torch.Tensor:
    """Integers in [0, n) (n int or int64 tensor); modulo of 53 hashed bits."""
    r = _lsr(hash_u64(seed, tensor_id, index), 11)
    return r % n


def normal_f64(seed: int, tensor_id: int, index: torch.Tensor) -> torch.Tensor:
    """Standard normal (fp64) for each flat index (Box-Muller, cosine branch)."""
    r1 = _lsr(hash_u64(seed, tensor_id, index, 0), 11)
    r2 = _lsr(hash_u64(seed, tensor_id, index, 1), 11)
    u1 = (r1.to(torch.float64) + 1.0) * (1.0 / 9007199254740992.0)   # (0, 1]
    u2 = r2.to(torch.float64) * (1.0 / 9007199254740992.0)           # [0, 1)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def normal_tensor(seed: int, tensor_id: int, shape, dtype: torch.dtype,
                  device="cpu", chunk: int = 1 << 22) -> torch.Tensor:
    """Packed tensor of N(0,1) draws rounded to ``dtype`` (round to nearest even)."""
    n = 1
    for s in shape:
        n *= int(s)
    out = torch.empty(n, dtype=dtype, device=device)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        out[lo:hi] = normal_f64(seed, tensor_id, idx).to(dtype)
    return out.view(*shape)


def distinct_positions(seed: int, tensor_id: int, stream: int, n_total: int, n_pick: int,
                       device="cpu") -> torch.Tensor:
    """``n_pick`` distinct positions in [0, n_total): ranks of hashed keys (no replacement)."""
    idx = torch.arange(n_total, dtype=torch.int64, device=device) + stream * n_total
    keys = _lsr(hash_u64(seed, tensor_id, idx), 1)          # non-negative, distinct w.h.p.
    order = torch.argsort(keys, stable=True)
    return torch.sort(order[:n_pick]).values


@dataclass(frozen=True)
class Workload:
    """Shape, budget and structure of one benchmark configuration."""
    name: str
    batch: int
    q_len: int
    kv_len: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                 # "f32" | "bf16"
    k_sel: int                 # global tokens chosen outside the window
    window: int                # forced most-recent tokens (query's own token included)
    n_sparse_layers: int
    structure: str             # "plain" | "needles_stratified" | "needles_uniform" | "clusters" | "decode_needles"
    seed: int
    n_needles: int = 32
    n_clusters: int = 64
    cluster_noise: float = 0.3

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


def _wl(c, **kw) -> Workload:
    return Workload(seed=BASE_SEED + c, **kw)


CONFIGS: Dict[str, Workload] = {
    # the five benchmark configurations
    "cfg1": _wl(1, name="cfg1", batch=1, q_len=512, kv_len=512, n_q_heads=4, n_kv_heads=1, head_dim=64,
                dtype="f32", k_sel=64, window=16, n_sparse_layers=1, structure="plain"),
    "cfg2": _wl(2, name="cfg2", batch=1, q_len=8192, kv_len=8192, n_q_heads=32, n_kv_heads=4, head_dim=128,
                dtype="bf16", k_sel=1024, window=128, n_sparse_layers=1, structure="needles_stratified"),
    "cfg3": _wl(3, name="cfg3", batch=2, q_len=32768, kv_len=32768, n_q_heads=32, n_kv_heads=4, head_dim=128,
                dtype="bf16", k_sel=2048, window=128, n_sparse_layers=3, structure="needles_uniform"),
    "cfg4": _wl(4, name="cfg4", batch=1, q_len=131072, kv_len=131072, n_q_heads=32, n_kv_heads=4, head_dim=128,
                dtype="bf16", k_sel=4096, window=256, n_sparse_layers=3, structure="clusters"),
    "cfg5": _wl(5, name="cfg5", batch=64, q_len=1, kv_len=65536, n_q_heads=32, n_kv_heads=4, head_dim=128,
                dtype="bf16", k_sel=2048, window=128, n_sparse_layers=1, structure="decode_needles"),
}


# The attention shape of the paper's own models (Table 1): multi-query attention, 64 query heads sharing one KV head,
# head_dim 256, 1024 selected + 128 window tokens.  Not benchmark configurations: measured beside them.
NATIVE: Dict[str, Workload] = {
    "native8k": _wl(11, name="native8k", batch=1, q_len=8192, kv_len=8192, n_q_heads=64, n_kv_heads=1, head_dim=256,
                    dtype="bf16", k_sel=1024, window=128, n_sparse_layers=3, structure="needles_stratified"),
    "native_decode": _wl(12, name="native_decode", batch=64, q_len=1, kv_len=65536, n_q_heads=64, n_kv_heads=1,
                         head_dim=256, dtype="bf16", k_sel=1024, window=128, n_sparse_layers=3,
                         structure="decode_needles"),
}


def scaled(name: str, **overrides) -> Workload:
    """A benchmark configuration with some fields replaced (small parity cases)."""
    return replace(CONFIGS[name], **overrides)


@dataclass
class Inputs:
    wl: Workload
    q_full: torch.Tensor                    # [B, Lq, Hq, D]  queries of the full-attention layer
    k: torch.Tensor                         # [B, Lk, Hkv, D] shared KV cache of the block
    v: torch.Tensor                         # [B, Lk, Hkv, D]
    q_sparse: List[torch.Tensor] = field(default_factory=list)   # one [B, Lq, Hq, D] per sparse layer
    needle_pos: Optional[torch.Tensor] = None                    # [B, Hkv, n_needles] (structure draws)


def _plant_needles(wl: Workload, q_full: torch.Tensor, k: torch.Tensor, device) -> torch.Tensor:
    """Overwrite needle key rows with 4x the (raw) query vector of a drawn target.

    K[b, p_n, g, :] = 4 * Q_full[b, t_n, h_n, :]: the needle has a logit of about
    4*sqrt(D) at its target query and N(0, 16) everywhere else.
    """
    B, Lq, Lk, Hkv, G, N = wl.batch, wl.q_len, wl.kv_len, wl.n_kv_heads, wl.group, wl.n_needles
    pos_all = torch.empty(B, Hkv, N, dtype=torch.int64, device=device)
    q_off = Lk - Lq                                           # absolute position of query 0
    for b in range(B):
        for g in range(Hkv):
            stream = b * Hkv + g
            if wl.structure == "needles_stratified":
                n = torch.arange(N, dtype=torch.int64, device=device)
                pos = n * (Lk // N) + Lk // (2 * N)
            else:
                pos = distinct_positions(wl.seed, TID_NEEDLE_POS, stream, Lk, N, device)
            ctr = torch.arange(N, dtype=torch.int64, device=device) + stream * N
            if wl.structure == "decode_needles":
                tgt = torch.zeros(N, dtype=torch.int64, device=device)       # the single decode query
            else:
                lo = torch.clamp(pos - q_off, min=0)                         # first query that sees the needle
                tgt = lo + uniform_int(wl.seed, TID_NEEDLE_TGT, ctr, Lq - lo)
            head = g * G + uniform_int(wl.seed, TID_NEEDLE_HEAD, ctr, G)
            rows = q_full[b, tgt, head, :].to(torch.float32) * 4.0
            k[b, pos, g, :] = rows.to(k.dtype)
            pos_all[b, g] = pos
    return pos_all


def _cluster_keys(wl: Workload, device, chunk_tokens: int = 1 << 15) -> torch.Tensor:
    """K[b, j, g, :] = centre[g, m(b, j, g)] + noise * N(0, I); centres ~ N(0, I_D)."""
    B, Lk, Hkv, D, C = wl.batch, wl.kv_len, wl.n_kv_heads, wl.head_dim, wl.n_clusters
    cidx = torch.arange(Hkv * C * D, dtype=torch.int64, device=device)
    centres = normal_f64(wl.seed, TID_CENTRES, cidx).view(Hkv, C, D)
    k = torch.empty(B, Lk, Hkv, D, dtype=wl.torch_dtype, device=device)
    garange = torch.arange(Hkv, dtype=torch.int64, device=device)
    for b in range(B):
        for lo in range(0, Lk, chunk_tokens):
            hi = min(Lk, lo + chunk_tokens)
            tok = torch.arange(lo, hi, dtype=torch.int64, device=device)
            row = (b * Lk + tok)[:, None] * Hkv + garange[None, :]            # [T, Hkv] flat row id
            m = uniform_int(wl.seed, TID_CLUSTER_ID, row, C)                  # [T, Hkv]
            flat = row[:, :, None] * D + torch.arange(D, dtype=torch.int64, device=device)
            noise = normal_f64(wl.seed, TID_K, flat)                          # [T, Hkv, D]
            cen = centres[garange[None, :].expand_as(m), m]                   # [T, Hkv, D]
            k[b, lo:hi] = (cen + wl.cluster_noise * noise).to(wl.torch_dtype)
    return k


def make_inputs(wl: Workload, device="cpu", n_sparse_layers: Optional[int] = None) -> Inputs:
    """Draw Q (full layer), the shared K/V cache and one Q per sparse layer."""
    dt = wl.torch_dtype
    qshape = (wl.batch, wl.q_len, wl.n_q_heads, wl.head_dim)
    kshape = (wl.batch, wl.kv_len, wl.n_kv_heads, wl.head_dim)
    q_full = normal_tensor(wl.seed, TID_Q_FULL, qshape, dt, device)
    v = normal_tensor(wl.seed, TID_V, kshape, dt, device)
    needle_pos = None
    if wl.structure == "clusters":
        k = _cluster_keys(wl, device)
    else:
        k = normal_tensor(wl.seed, TID_K, kshape, dt, device)
        if wl.structure != "plain":
            needle_pos = _plant_needles(wl, q_full, k, device)
    nl = wl.n_sparse_layers if n_sparse_layers is None else n_sparse_layers
    q_sparse = [normal_tensor(wl.seed, TID_Q_SPARSE0 + l, qshape, dt, device) for l in range(nl)]
    return Inputs(wl, q_full, k, v, q_sparse, needle_pos)


def sample_rows(wl: Workload, n_rows: int = 64) -> List[int]:
    """Query rows checked one by one at sizes where the oracle cannot do them all.

    The budget edges {0, w-1, w, w+k-1, w+k, Lq-1} plus seeded-uniform rows.
    """
    Lq = wl.q_len
    edges = [0, wl.window - 1, wl.window, wl.window + wl.k_sel - 1, wl.window + wl.k_sel, Lq - 1]
    rows = sorted({r for r in edges if 0 <= r < Lq})
    ctr = torch.arange(4 * n_rows, dtype=torch.int64)
    extra = uniform_int(wl.seed, 200, ctr, Lq).tolist()
    for r in extra:
        if len(rows) >= min(n_rows, Lq):
            break
        if r not in rows:
            rows.append(r)
    return sorted(rows)


def quantize_kv_e4m3(x: torch.Tensor):
    """Stand-in for the producer of an FP8 KV cache (outside the attention path): one fp32 scale per (token, KV head)
    = amax / 448 (1 for an all-zero row), codes = x / scale rounded to the nearest e4m3 value by torch's own cast.
    Returns ``(codes uint8 [B, L, Hkv, D], scales fp32 [B, L, Hkv])``."""
    xf = x.float()
    amax = xf.abs().amax(dim=-1)
    scale = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax)).float()
    y = (xf / scale[..., None]).clamp(-448.0, 448.0).to(torch.float8_e4m3fn)
    return y.view(torch.uint8).contiguous(), scale.contiguous()
