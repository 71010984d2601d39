"""ctypes front end of the CPU oracle (``hs2_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never import it.

Tensors are numpy arrays: fp32 as ``float32``, bf16 as ``uint16`` bit patterns, packed
``[B, L, H, D]``.  Results are fp64.
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hs2_oracle.c")
_LIB = os.path.join(_HERE, "libhs2_oracle.so")

AGG_MAX_PROB, AGG_MAX_LOGIT, AGG_SUM_PROB = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP only spreads whole rows over threads)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Problem(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("q_len", C.c_int32), ("kv_len", C.c_int32),
                ("k_sel", C.c_int32), ("window", C.c_int32), ("scale", C.c_double),
                ("dtype", C.c_int32), ("agg", C.c_int32),
                ("q_start", C.c_void_p), ("kv_lens", C.c_void_p)]


_lib = None


def _get():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.hs2o_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(_get().hs2o_num_threads())


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _as_input(x) -> Tuple[np.ndarray, int]:
    """numpy view of an input tensor: float32 -> dtype 0, uint16 (bf16 bits) -> dtype 1.

    torch tensors (CPU) are accepted for convenience and viewed without a copy.
    """
    if not isinstance(x, np.ndarray):
        import torch
        x = x.detach().contiguous()
        if x.dtype == torch.bfloat16:
            x = x.view(torch.int16).numpy().view(np.uint16)
        else:
            x = x.numpy()
    x = np.ascontiguousarray(x)
    if x.dtype == np.float32:
        return x, 0
    if x.dtype == np.uint16:
        return x, 1
    raise TypeError("oracle inputs are float32 or bf16 bit patterns (uint16), got %s" % x.dtype)


class Problem:
    """Shapes and budgets of one call (mirrors the library's problem statement)."""

    def __init__(self, q, k, k_sel: int, window: int, scale: Optional[float] = None,
                 q_start: Optional[Sequence[int]] = None, kv_lens: Optional[Sequence[int]] = None,
                 agg: int = AGG_MAX_PROB):
        self.q, dq = _as_input(q)
        self.k, dk = _as_input(k)
        assert dq == dk and self.q.ndim == 4 and self.k.ndim == 4
        B, Lq, Hq, D = self.q.shape
        Bk, Lk, Hkv, Dk = self.k.shape
        assert B == Bk and D == Dk and Hq % Hkv == 0
        self.shape = (B, Lq, Lk, Hq, Hkv, D)
        self.k_sel, self.window = int(k_sel), int(window)
        self.q_start = None if q_start is None else np.ascontiguousarray(q_start, dtype=np.int32)
        self.kv_lens = None if kv_lens is None else np.ascontiguousarray(kv_lens, dtype=np.int32)
        self.c = _Problem(B, Hq, Hkv, D, Lq, Lk, self.k_sel, self.window,
                          float(scale) if scale else 1.0 / math.sqrt(D), dq, agg,
                          _ptr(self.q_start), _ptr(self.kv_lens))

    def pos(self, b: int, i: int) -> int:
        kvl = self.shape[2] if self.kv_lens is None else int(self.kv_lens[b])
        q0 = kvl - self.shape[1] if self.q_start is None else int(self.q_start[b])
        return q0 + i

    def kvlen(self, b: int) -> int:
        return self.shape[2] if self.kv_lens is None else int(self.kv_lens[b])


def _rows(prob: Problem, rows):
    if rows is None:
        B, Lq = prob.shape[0], prob.shape[1]
        rows = [(b, i) for b in range(B) for i in range(Lq)]
    rb = np.ascontiguousarray([r[0] for r in rows], dtype=np.int32)
    ri = np.ascontiguousarray([r[1] for r in rows], dtype=np.int32)
    return rb, ri


def full_attn_select(q, k, v, k_sel, window, rows=None, scale=None, q_start=None, kv_lens=None,
                     agg=AGG_MAX_PROB, want_idx=True, want_scores=False):
    """Full causal attention + selection for the listed (b, i) rows (all rows when None).

    Returns ``(O [n,Hq,D], LSE [n,Hq], idx [n,Hkv,k] | None, scores [n,Hkv,Lk] | None)``;
    scores are the aggregated selection scores (probabilities unless ``agg`` says logits),
    ``-inf`` for keys the query cannot see.
    """
    prob = Problem(q, k, k_sel, window, scale, q_start, kv_lens, agg)
    vv, _ = _as_input(v)
    B, Lq, Lk, Hq, Hkv, D = prob.shape
    rb, ri = _rows(prob, rows)
    n = len(rb)
    O = np.zeros((n, Hq, D), dtype=np.float64)
    LSE = np.zeros((n, Hq), dtype=np.float64)
    idx = np.full((n, Hkv, k_sel), -1, dtype=np.int32) if want_idx else None
    sc = np.zeros((n, Hkv, Lk), dtype=np.float64) if want_scores else None
    _get().hs2o_full_attn_select_rows(C.byref(prob.c), _ptr(prob.q), _ptr(prob.k), _ptr(vv), C.c_int(n),
                                      _ptr(rb), _ptr(ri), _ptr(O), _ptr(LSE), _ptr(idx), _ptr(sc))
    return O, LSE, idx, sc


def select(scores, pos, kvlen, window: int, k_sel: int) -> np.ndarray:
    """Top-k outside the window on given scores ``[n, Lk]`` (any float dtype) -> idx ``[n, k]``."""
    sc = np.ascontiguousarray(scores, dtype=np.float64)
    n, Lk = sc.shape
    pos = np.ascontiguousarray(np.broadcast_to(np.asarray(pos, dtype=np.int32), (n,)))
    kvlen = np.ascontiguousarray(np.broadcast_to(np.asarray(kvlen, dtype=np.int32), (n,)))
    idx = np.full((n, k_sel), -1, dtype=np.int32)
    _get().hs2o_select_rows(_ptr(sc), C.c_int(Lk), C.c_int(n), _ptr(pos), _ptr(kvlen),
                            C.c_int(window), C.c_int(k_sel), _ptr(idx))
    return idx


def sparse_attn(q, k, v, idx, window, rows=None, sink=None, scale=None, q_start=None, kv_lens=None,
                want_member=False, gate=None):
    """Sparse attention over (valid idx) U window for the listed rows.

    ``idx`` is ``[n, Hkv, k]`` aligned with ``rows``.  Returns ``(O [n,Hq,D], LSE [n,Hq], member)``.
    ``gate`` (``[B, Lq, Hq, D]`` logits, optional) is the sigmoid output gate of the sparse layers
    (Section 4.1): the attention output of a row is multiplied elementwise by 1 / (1 + exp(-gate)).
    """
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    k_sel = idx.shape[-1]
    prob = Problem(q, k, k_sel, window, scale, q_start, kv_lens)
    vv, _ = _as_input(v)
    B, Lq, Lk, Hq, Hkv, D = prob.shape
    rb, ri = _rows(prob, rows)
    n = len(rb)
    assert idx.shape == (n, Hkv, k_sel), (idx.shape, (n, Hkv, k_sel))
    O = np.zeros((n, Hq, D), dtype=np.float64)
    LSE = np.zeros((n, Hq), dtype=np.float64)
    member = np.zeros((n, Hkv, Lk), dtype=np.uint8) if want_member else None
    sk = None if sink is None else np.ascontiguousarray(sink, dtype=np.float64)
    _get().hs2o_sparse_attn_rows(C.byref(prob.c), _ptr(prob.q), _ptr(prob.k), _ptr(vv), _ptr(idx), _ptr(sk),
                                 C.c_int(n), _ptr(rb), _ptr(ri), _ptr(O), _ptr(LSE), _ptr(member))
    if gate is not None:
        gg, code = _as_input(gate)                  # the exact input values, widened to fp64
        if code == 1:                               # bf16 bit patterns: the upper half of an fp32
            gg = (gg.astype(np.uint32) << 16).view(np.float32)
        gg = gg.astype(np.float64).reshape(B, Lq, Hq, D)
        O = O * (1.0 / (1.0 + np.exp(-gg[rb, ri])))
    return O, LSE, member


def decode_e4m3(codes):
    """Value of every e4m3 code, from the format's definition: 1 sign bit, 4 exponent bits (bias 7), 3 mantissa
    bits; exponent field 0 is subnormal (mantissa / 8 * 2^-6); there are no infinities, S.1111.111 is NaN."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 0x7).astype(np.float64)
    val = np.where(e == 0, m / 8.0 * 2.0 ** -6, (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64)))
    val = np.where((e == 15) & ((c & 0x7) == 7), np.nan, val)
    return sign * val


def dequant_e4m3(codes, scales):
    """FP8 cache contents: code value times the scale of its (token, KV head), as an fp32 array (the cache value is
    defined as that product rounded to fp32)."""
    if not isinstance(codes, np.ndarray):
        codes = codes.detach().cpu().numpy()
    if not isinstance(scales, np.ndarray):
        scales = scales.detach().cpu().numpy()
    return (decode_e4m3(codes) * scales.astype(np.float64)[..., None]).astype(np.float32)


def select_blocks(scores, pos, kvlen, window: int, k_sel: int, block: int) -> np.ndarray:
    """Block-level selection (the variant of the paper's first ablation, Section 5) on given scores ``[n, Lk]``.

    The candidates of a row are the keys 0 .. min(pos - window, kvlen - 1); they are cut into aligned blocks of
    ``block`` keys (the last may be partial); a block scores the maximum over its candidates; the ``k_sel // block``
    best blocks (ties: lower block first) are kept and their candidate keys listed ascending, -1 padded.
    """
    sc = np.asarray(scores, dtype=np.float64)
    n, Lk = sc.shape
    pos = np.broadcast_to(np.asarray(pos, dtype=np.int64), (n,))
    kvlen = np.broadcast_to(np.asarray(kvlen, dtype=np.int64), (n,))
    assert block >= 1 and k_sel % block == 0
    idx = np.full((n, k_sel), -1, dtype=np.int32)
    for r in range(n):
        nk = int(max(0, min(pos[r] - window + 1, kvlen[r])))
        nb = (nk + block - 1) // block
        best = [max(sc[r, m * block:min(nk, (m + 1) * block)]) for m in range(nb)]
        order = sorted(range(nb), key=lambda m: (-best[m], m))[:k_sel // block]
        keys = [j for m in sorted(order) for j in range(m * block, min(nk, (m + 1) * block))]
        idx[r, :len(keys)] = keys
    return idx


def kv_project(h, w):
    """KV-cache producer (Section 3.2, KV Bridging: K = Proj^K(H), V = Proj^V(H)): ``H [T, dm] @ W [N, dm]^T`` in fp64 on
    the exact input values."""
    def f64(x):
        a, code = _as_input(x)
        if code == 1:
            a = (a.astype(np.uint32) << 16).view(np.float32)
        return a.astype(np.float64)
    return f64(h) @ f64(w).T
