"""Thin ctypes binding of ``libhs2.so``: argument marshalling only.

Every step of the path runs inside the CUDA library; this module turns torch tensors into
device pointers, fills the ``hs2_problem`` struct, allocates outputs / scratch with torch when the
caller did not pass them, and raises on a non-zero status.  There is no fallback: a missing
library or a missing GPU is an error.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libhs2.so")

HS2_OK, HS2_ERR_INVALID_ARG, HS2_ERR_UNSUPPORTED, HS2_ERR_WORKSPACE_TOO_SMALL, HS2_ERR_CUDA, \
    HS2_ERR_STATIC_SCRATCH = range(6)
HS2_STATIC_DECODE_MAX_PAIRS = 64
HS2_F32, HS2_BF16 = 0, 1
HS2_OP_FULL_ATTN_SELECT, HS2_OP_TOPK_SELECT, HS2_OP_SPARSE_ATTN_PREFILL, HS2_OP_SPARSE_ATTN_DECODE = range(4)
HS2_OP_FULL_ATTN_SELECT_FP8KV = 4

EXPORTS = ["hs2_workspace_bytes", "hs2_full_attn_select", "hs2_topk_select", "hs2_sparse_attn_prefill",
           "hs2_sparse_attn_decode", "hs2_sparse_attn_prefill_gated", "hs2_sparse_attn_decode_gated",
           "hs2_sparse_attn_prefill_fp8kv", "hs2_sparse_attn_decode_fp8kv", "hs2_full_attn_select_fp8kv", "hs2_kv_project",
           "hs2_kv_project_fp8_records",
           "hs2_sparse_attn_decode_static", "hs2_probe_gather", "hs2_status_string", "hs2_last_cuda_error",
           "hs2_launch_count", "hs2_device_error_flags", "hs2_set_filter_min_keys", "hs2_set_tcgen05_enabled"]


class HS2Error(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__("%s: %s%s" % (where, hs2_status_string(status), detail))


class _CProblem(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("q_len", C.c_int32), ("kv_len", C.c_int32),
                ("k_sel", C.c_int32), ("window", C.c_int32), ("softmax_scale", C.c_float),
                ("dtype", C.c_int), ("q_start", C.c_void_p), ("kv_lens", C.c_void_p),
                ("q_stride", C.c_int64 * 3), ("kv_stride", C.c_int64 * 3), ("o_stride", C.c_int64 * 3),
                ("select_block", C.c_int32), ("kv_scale_stride", C.c_int64 * 3)]


_lib = None


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """dlopen the in-tree library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError("%s is missing: build it with `python -m paper_2609_26368_b200.build`" % _LIB_PATH)
        lib = C.CDLL(_LIB_PATH)
        lib.hs2_workspace_bytes.restype = C.c_size_t
        lib.hs2_workspace_bytes.argtypes = [C.POINTER(_CProblem), C.c_int]
        lib.hs2_status_string.restype = C.c_char_p
        lib.hs2_status_string.argtypes = [C.c_int]
        lib.hs2_last_cuda_error.restype = C.c_int
        lib.hs2_launch_count.restype = C.c_ulonglong
        vp, sz = C.c_void_p, C.c_size_t
        pp = C.POINTER(_CProblem)
        lib.hs2_full_attn_select.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.hs2_topk_select.argtypes = [pp, vp, vp, vp, sz, vp]
        lib.hs2_sparse_attn_prefill.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.hs2_sparse_attn_decode.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.hs2_sparse_attn_decode_static.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.hs2_sparse_attn_prefill_gated.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.hs2_sparse_attn_decode_gated.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.hs2_kv_project.argtypes = [C.c_int64, C.c_int32, C.c_int32, vp, C.c_int64, vp, C.c_int64, vp, C.c_int64, vp, vp]
        lib.hs2_kv_project.restype = C.c_int
        lib.hs2_kv_project_fp8_records.argtypes = [C.c_int64, C.c_int32, C.c_int32, vp, C.c_int64, vp, C.c_int64, vp, C.c_int64,
                                                   C.c_int64, vp, C.c_int64, C.c_int64, vp]
        lib.hs2_kv_project_fp8_records.restype = C.c_int
        lib.hs2_sparse_attn_prefill_fp8kv.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.hs2_sparse_attn_decode_fp8kv.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.hs2_full_attn_select_fp8kv.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.hs2_probe_gather.argtypes = [pp, vp, vp, vp, C.c_int, vp, vp]
        lib.hs2_probe_gather.restype = C.c_int
        for f in ("hs2_full_attn_select", "hs2_topk_select", "hs2_sparse_attn_prefill", "hs2_sparse_attn_decode",
                  "hs2_sparse_attn_prefill_gated", "hs2_sparse_attn_decode_gated", "hs2_sparse_attn_decode_static",
                  "hs2_sparse_attn_prefill_fp8kv", "hs2_sparse_attn_decode_fp8kv"):
            getattr(lib, f).restype = C.c_int
        _lib = lib
    return _lib


def hs2_device_error_flags() -> int:
    """Device error word of the library (0 = fine); synchronises the device."""
    v = C.c_uint(0)
    _check(load_library().hs2_device_error_flags(C.byref(v)), "hs2_device_error_flags")
    return int(v.value)


def hs2_set_filter_min_keys(min_keys: int) -> int:
    """Tuning knob: kv_len from which the full layer's selection uses filtered candidate lists; returns the old value."""
    return int(load_library().hs2_set_filter_min_keys(int(min_keys)))


def hs2_set_tcgen05_enabled(enabled: int) -> int:
    """Testing knob: 0 routes the full layer through its mma.sync kernels; returns the previous setting."""
    return int(load_library().hs2_set_tcgen05_enabled(int(enabled)))


def hs2_launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(load_library().hs2_launch_count())


def hs2_status_string(status: int) -> str:
    return load_library().hs2_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != HS2_OK:
        detail = ""
        if status == HS2_ERR_CUDA:
            detail = " (cudaError %d)" % load_library().hs2_last_cuda_error()
        raise HS2Error(status, where, detail)


def _dp(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _strides(t: torch.Tensor):
    assert t.stride(3) == 1, "last dimension must be contiguous"
    return (C.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2))


class Problem:
    """Host-side description of one call; mirrors ``hs2_problem``."""

    def __init__(self, batch, q_len, kv_len, n_q_heads, n_kv_heads, head_dim, k_sel, window, dtype=torch.bfloat16,
                 softmax_scale: float = 0.0, q_start: Optional[torch.Tensor] = None,
                 kv_lens: Optional[torch.Tensor] = None, select_block: int = 0):
        self.batch, self.q_len, self.kv_len = int(batch), int(q_len), int(kv_len)
        self.n_q_heads, self.n_kv_heads, self.head_dim = int(n_q_heads), int(n_kv_heads), int(head_dim)
        self.k_sel, self.window = int(k_sel), int(window)
        self.dtype = dtype
        self.softmax_scale = float(softmax_scale)
        self.q_start, self.kv_lens = q_start, kv_lens
        self.select_block = int(select_block)
        for t in (q_start, kv_lens):
            assert t is None or (t.dtype == torch.int32 and t.is_cuda and t.is_contiguous())

    @classmethod
    def from_tensors(cls, q, k, k_sel, window, **kw):
        B, Lq, Hq, D = q.shape
        _, Lk, Hkv, _ = k.shape
        return cls(B, Lq, Lk, Hq, Hkv, D, k_sel, window, dtype=q.dtype, **kw)

    def c_struct(self, q=None, kv=None, o=None) -> _CProblem:
        if self.dtype not in (torch.float32, torch.bfloat16):
            raise TypeError("hs2 tensors are float32 or bfloat16")
        c = _CProblem(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.q_len, self.kv_len,
                      self.k_sel, self.window, self.softmax_scale,
                      HS2_F32 if self.dtype == torch.float32 else HS2_BF16,
                      None if self.q_start is None else self.q_start.data_ptr(),
                      None if self.kv_lens is None else self.kv_lens.data_ptr())
        c.select_block = self.select_block
        if q is not None:
            c.q_stride = _strides(q)
        if kv is not None:
            c.kv_stride = _strides(kv)
        if o is not None:
            c.o_stride = _strides(o)
        return c


def hs2_workspace_bytes(prob: Problem, op: int) -> int:
    c = prob.c_struct()
    return int(load_library().hs2_workspace_bytes(C.byref(c), int(op)))


def _workspace(prob: Problem, op: int, device, ws: Optional[torch.Tensor]):
    if ws is not None:
        return ws
    n = hs2_workspace_bytes(prob, op)
    return torch.empty(max(n, 256), dtype=torch.uint8, device=device)


def _check_inputs(prob: Problem, q, k, v):
    assert q.is_cuda and k.is_cuda and v.is_cuda, "hs2 runs on CUDA tensors only"
    assert q.dtype == k.dtype == v.dtype == prob.dtype
    assert tuple(q.shape) == (prob.batch, prob.q_len, prob.n_q_heads, prob.head_dim)
    assert tuple(k.shape) == tuple(v.shape) == (prob.batch, prob.kv_len, prob.n_kv_heads, prob.head_dim)
    assert k.stride() == v.stride(), "K and V share one stride triple"


def hs2_full_attn_select(prob: Problem, q, k, v, *, out=None, lse=None, idx=None, want_idx=True,
                         scores_dbg=None, want_scores=False, ws=None, stream=None):
    """FA layer: returns ``(O, LSE, idx | None, scores_dbg | None)``."""
    _check_inputs(prob, q, k, v)
    dev = q.device
    out = torch.empty_like(q) if out is None else out
    lse = torch.empty(prob.batch, prob.n_q_heads, prob.q_len, dtype=torch.float32, device=dev) if lse is None else lse
    if idx is None and want_idx:
        idx = torch.empty(prob.batch, prob.n_kv_heads, prob.q_len, prob.k_sel, dtype=torch.int32, device=dev)
    if scores_dbg is None and want_scores:
        scores_dbg = torch.empty(prob.batch, prob.n_kv_heads, prob.q_len, prob.kv_len, dtype=torch.float32, device=dev)
    if idx is not None and scores_dbg is None:
        ws = _workspace(prob, HS2_OP_FULL_ATTN_SELECT, dev, ws)
    c = prob.c_struct(q, k, out)
    st = load_library().hs2_full_attn_select(C.byref(c), _dp(q), _dp(k), _dp(v), _dp(out), _dp(lse), _dp(idx),
                                             _dp(scores_dbg), _dp(ws), 0 if ws is None else ws.numel(), _stream(stream))
    _check(st, "hs2_full_attn_select")
    return out, lse, idx, scores_dbg


def hs2_topk_select(prob: Problem, scores, *, idx=None, stream=None):
    """Token-level top-k outside the window on a float32 score tensor ``[B, Hkv, Lq, Lk]``."""
    assert scores.is_cuda and scores.dtype == torch.float32 and scores.is_contiguous()
    assert tuple(scores.shape) == (prob.batch, prob.n_kv_heads, prob.q_len, prob.kv_len)
    if idx is None:
        idx = torch.empty(prob.batch, prob.n_kv_heads, prob.q_len, prob.k_sel, dtype=torch.int32, device=scores.device)
    c = prob.c_struct()
    st = load_library().hs2_topk_select(C.byref(c), _dp(scores), _dp(idx), None, 0, _stream(stream))
    _check(st, "hs2_topk_select")
    return idx


def _sparse(fn_name, op, prob, q, k, v, idx, sink, out, lse, want_lse, ws, stream, gate=None):
    _check_inputs(prob, q, k, v)
    dev = q.device
    if idx is not None:
        assert idx.dtype == torch.int32 and idx.is_contiguous() and idx.is_cuda
        assert tuple(idx.shape) == (prob.batch, prob.n_kv_heads, prob.q_len, prob.k_sel)
    if sink is not None:
        assert sink.dtype == torch.float32 and sink.is_cuda and sink.numel() == prob.n_q_heads
    out = torch.empty_like(q) if out is None else out
    if lse is None and want_lse:
        lse = torch.empty(prob.batch, prob.n_q_heads, prob.q_len, dtype=torch.float32, device=dev)
    ws = _workspace(prob, op, dev, ws)
    c = prob.c_struct(q, k, out)
    if gate is not None:   # the gated entry point: gate logits laid out like the output
        assert gate.is_cuda and gate.dtype == out.dtype and gate.shape == out.shape and gate.stride() == out.stride()
        fn_name += "_gated"
        st = getattr(load_library(), fn_name)(C.byref(c), _dp(q), _dp(k), _dp(v), _dp(idx), _dp(sink), _dp(gate), _dp(out),
                                              _dp(lse), _dp(ws), ws.numel(), _stream(stream))
    else:
        st = getattr(load_library(), fn_name)(C.byref(c), _dp(q), _dp(k), _dp(v), _dp(idx), _dp(sink), _dp(out), _dp(lse),
                                              _dp(ws), ws.numel(), _stream(stream))
    _check(st, fn_name)
    return out, lse


def hs2_sparse_attn_prefill(prob: Problem, q, k, v, idx, *, sink=None, gate=None, out=None, lse=None, want_lse=False,
                            ws=None, stream=None):
    """SA layer, prefill: attention over (idx) U (forced window); returns ``(O, LSE | None)``.
    With ``gate`` (logits shaped like the output) the output is multiplied by sigmoid(gate) in the kernel's store."""
    return _sparse("hs2_sparse_attn_prefill", HS2_OP_SPARSE_ATTN_PREFILL, prob, q, k, v, idx, sink, out, lse,
                   want_lse, ws, stream, gate)


def hs2_sparse_attn_decode(prob: Problem, q, k, v, idx, *, sink=None, gate=None, out=None, lse=None, want_lse=False,
                           ws=None, stream=None):
    """SA layer, decode (q_len == 1, split over the attended set); returns ``(O, LSE | None)``."""
    return _sparse("hs2_sparse_attn_decode", HS2_OP_SPARSE_ATTN_DECODE, prob, q, k, v, idx, sink, out, lse,
                   want_lse, ws, stream, gate)


def _sparse_fp8(fn_name, prob, q, k8, v8, k_scale, v_scale, idx, sink, out, lse, want_lse, stream):
    assert q.is_cuda and q.dtype == torch.bfloat16 and q.stride(-1) == 1
    for t in (k8, v8):
        assert t.is_cuda and t.dtype == torch.uint8 and t.stride(-1) == 1
        assert tuple(t.shape) == (prob.batch, prob.kv_len, prob.n_kv_heads, prob.head_dim)
    assert k8.stride() == v8.stride()
    for t in (k_scale, v_scale):
        assert t.is_cuda and t.dtype == torch.float32
        assert tuple(t.shape) == (prob.batch, prob.kv_len, prob.n_kv_heads)
    assert k_scale.stride() == v_scale.stride()   # may be views into records that also hold the codes
    if idx is not None:
        assert idx.dtype == torch.int32 and idx.is_contiguous() and idx.is_cuda
        assert tuple(idx.shape) == (prob.batch, prob.n_kv_heads, prob.q_len, prob.k_sel)
    if sink is not None:
        assert sink.dtype == torch.float32 and sink.is_cuda and sink.numel() == prob.n_q_heads
    out = torch.empty_like(q) if out is None else out
    if lse is None and want_lse:
        lse = torch.empty(prob.batch, prob.n_q_heads, prob.q_len, dtype=torch.float32, device=q.device)
    c = prob.c_struct(q, k8, out)
    c.kv_scale_stride = (C.c_int64 * 3)(*k_scale.stride())
    st = getattr(load_library(), fn_name)(C.byref(c), _dp(q), _dp(k8), _dp(v8), _dp(k_scale), _dp(v_scale), _dp(idx),
                                          _dp(sink), _dp(out), _dp(lse), _stream(stream))
    _check(st, fn_name)
    return out, lse


def hs2_full_attn_select_fp8kv(prob: Problem, q, k8, v8, k_scale, v_scale, *, out=None, lse=None, idx=None, want_idx=True,
                               ws=None, stream=None):
    """FA layer, decode step (one query per sequence), on an e4m3 cache: returns ``(O, LSE, idx | None)``."""
    assert q.is_cuda and q.dtype == torch.bfloat16 and q.stride(-1) == 1
    for t in (k8, v8):
        assert t.is_cuda and t.dtype == torch.uint8 and t.stride(-1) == 1
        assert tuple(t.shape) == (prob.batch, prob.kv_len, prob.n_kv_heads, prob.head_dim)
    assert k8.stride() == v8.stride()
    for t in (k_scale, v_scale):
        assert t.is_cuda and t.dtype == torch.float32
        assert tuple(t.shape) == (prob.batch, prob.kv_len, prob.n_kv_heads)
    assert k_scale.stride() == v_scale.stride()   # may be views into records that also hold the codes
    dev = q.device
    out = torch.empty_like(q) if out is None else out
    lse = torch.empty(prob.batch, prob.n_q_heads, prob.q_len, dtype=torch.float32, device=dev) if lse is None else lse
    if idx is None and want_idx:
        idx = torch.empty(prob.batch, prob.n_kv_heads, prob.q_len, prob.k_sel, dtype=torch.int32, device=dev)
    if idx is not None:
        ws = _workspace(prob, HS2_OP_FULL_ATTN_SELECT_FP8KV, dev, ws)
    c = prob.c_struct(q, k8, out)
    c.kv_scale_stride = (C.c_int64 * 3)(*k_scale.stride())
    st = load_library().hs2_full_attn_select_fp8kv(C.byref(c), _dp(q), _dp(k8), _dp(v8), _dp(k_scale), _dp(v_scale), _dp(out),
                                                   _dp(lse), _dp(idx), _dp(ws), 0 if ws is None else ws.numel(), _stream(stream))
    _check(st, "hs2_full_attn_select_fp8kv")
    return out, lse, idx


def hs2_sparse_attn_prefill_fp8kv(prob: Problem, q, k8, v8, k_scale, v_scale, idx, *, sink=None, out=None, lse=None,
                                  want_lse=False, stream=None):
    """SA layer, prefill, on an e4m3 cache (uint8 codes + fp32 scale per (token, KV head)); bf16 Q and O."""
    return _sparse_fp8("hs2_sparse_attn_prefill_fp8kv", prob, q, k8, v8, k_scale, v_scale, idx, sink, out, lse, want_lse,
                       stream)


def hs2_sparse_attn_decode_fp8kv(prob: Problem, q, k8, v8, k_scale, v_scale, idx, *, sink=None, out=None, lse=None,
                                 want_lse=False, stream=None):
    """SA layer, decode (q_len == 1), on an e4m3 cache."""
    return _sparse_fp8("hs2_sparse_attn_decode_fp8kv", prob, q, k8, v8, k_scale, v_scale, idx, sink, out, lse, want_lse,
                       stream)


def hs2_kv_project(h, w, *, out=None, fp8=False, scales=None, stream=None):
    """Cache producer: ``out[T, N] = h[T, dm] @ w[N, dm].T`` (bf16), or with ``fp8=True`` e4m3 codes (uint8) plus one
    fp32 scale per (token, 128 columns).  ``out`` may be a strided 2-D view (e.g. a slice of a fused cache).
    Returns ``out`` or ``(out, scales)``."""
    assert h.is_cuda and w.is_cuda and h.dtype == torch.bfloat16 and w.dtype == torch.bfloat16
    assert h.dim() == 2 and w.dim() == 2 and h.shape[1] == w.shape[1] and h.stride(1) == 1 and w.stride(1) == 1
    T, dm = h.shape
    N = w.shape[0]
    if out is None:
        out = torch.empty(T, N, dtype=torch.uint8 if fp8 else torch.bfloat16, device=h.device)
    assert out.dim() == 2 and tuple(out.shape) == (T, N) and out.stride(1) == 1
    assert out.dtype == (torch.uint8 if fp8 else torch.bfloat16)
    if fp8 and scales is None:
        scales = torch.empty(T, N // 128, dtype=torch.float32, device=h.device)
    st = load_library().hs2_kv_project(T, dm, N, _dp(h), h.stride(0), _dp(w), w.stride(0), _dp(out), out.stride(0),
                                       _dp(scales) if fp8 else None, _stream(stream))
    _check(st, "hs2_kv_project")
    return (out, scales) if fp8 else out


def hs2_kv_project_fp8_records(h, w, codes, scales, *, stream=None):
    """Cache producer writing e4m3 codes and scales into records: ``codes`` is a uint8 view ``[T, G, 128]`` (G column
    groups = heads of dim 128, any 16-byte-multiple strides between tokens and groups, the 128 codes contiguous),
    ``scales`` a float32 view ``[T, G]``; both may point into the same buffer.  Returns ``(codes, scales)``."""
    assert h.is_cuda and w.is_cuda and h.dtype == torch.bfloat16 and w.dtype == torch.bfloat16
    assert h.dim() == 2 and w.dim() == 2 and h.shape[1] == w.shape[1] and h.stride(1) == 1 and w.stride(1) == 1
    T, dm = h.shape
    N = w.shape[0]
    assert codes.dtype == torch.uint8 and tuple(codes.shape) == (T, N // 128, 128) and codes.stride(2) == 1
    assert scales.dtype == torch.float32 and tuple(scales.shape) == (T, N // 128)
    st = load_library().hs2_kv_project_fp8_records(T, dm, N, _dp(h), h.stride(0), _dp(w), w.stride(0), _dp(codes),
                                                   codes.stride(0), codes.stride(1), _dp(scales), scales.stride(0),
                                                   scales.stride(1), _stream(stream))
    _check(st, "hs2_kv_project_fp8_records")
    return codes, scales


def hs2_probe_gather(prob: Problem, k, v, idx, *, mode=0, sink_word=None, stream=None):
    """Measurement aid: only the K/V row fetches of ``hs2_sparse_attn_prefill`` on this problem (same items, same
    order, same validity rules), no arithmetic.  ``mode`` 0 loads past L1, 1 through it.  Returns ``sink_word``."""
    assert k.is_cuda and v.is_cuda and k.dtype == torch.bfloat16
    if sink_word is None:
        sink_word = torch.zeros(1, dtype=torch.int32, device=k.device)
    c = prob.c_struct(None, k, None)
    st = load_library().hs2_probe_gather(C.byref(c), _dp(k), _dp(v), _dp(idx), int(mode), _dp(sink_word), _stream(stream))
    _check(st, "hs2_probe_gather")
    return sink_word


def hs2_sparse_attn_decode_static(prob: Problem, q, k, v, idx, *, sink=None, out, lse=None, stream=None):
    """Decode for callers that may not allocate: the split kernel's partials live in a fixed
    8.5 MB array inside the library, so no workspace is passed and nothing is allocated - here
    included, which is why ``out`` (and ``lse``, if wanted) must be given.  Limit:
    ``batch * n_kv_heads <= 64`` for groups of up to 8 query heads per KV head, ``<= 32`` for groups of 16 (which
    run as two sub-groups of 8).  Calls on one device share that array: keep them ordered on the GPU.
    """
    _check_inputs(prob, q, k, v)
    assert out is not None and out.is_cuda and out.shape == q.shape and out.dtype == q.dtype
    if idx is not None:
        assert idx.dtype == torch.int32 and idx.is_contiguous() and idx.is_cuda
    c = prob.c_struct(q, k, out)
    st = load_library().hs2_sparse_attn_decode_static(C.byref(c), _dp(q), _dp(k), _dp(v), _dp(idx), _dp(sink),
                                                      _dp(out), _dp(lse), _stream(stream))
    _check(st, "hs2_sparse_attn_decode_static")
    return out, lse
