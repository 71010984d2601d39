"""Helpers shared by the GPU parity tests: run the CUDA library and the oracle on the same bytes.

Tolerances (stated by the benchmark definition): attention outputs max-abs 2e-2 and mean-abs 2e-3 for
bf16 I/O, 1e-4 for fp32; selection indices bit-exact on equal fp32 scores; end to end an index may
differ from the oracle's only where the oracle's scores are within 1e-3 relative of the row's
k-th largest score (|delta log A| <= 1e-3).
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

import oracle
import paper_2609_26368_b200 as hs2

TOL = {torch.float32: dict(max_abs=1e-4, mean_abs=1e-4, lse=1e-4, score=2e-4),
       torch.bfloat16: dict(max_abs=2e-2, mean_abs=2e-3, lse=2e-3, score=1e-3)}


def to_host(t: torch.Tensor) -> torch.Tensor:
    return t.detach().cpu().contiguous()


def assert_output_close(got: torch.Tensor, want: np.ndarray, dtype, what=""):
    g = got.detach().float().cpu().numpy().astype(np.float64)
    err = np.abs(g - want)
    tol = TOL[dtype]
    assert np.isfinite(g).all(), what + ": non-finite output"
    assert err.max() <= tol["max_abs"], "%s: max-abs %.3e > %.1e" % (what, err.max(), tol["max_abs"])
    assert err.mean() <= tol["mean_abs"], "%s: mean-abs %.3e > %.1e" % (what, err.mean(), tol["mean_abs"])


def rows_all(B: int, Lq: int) -> List[Tuple[int, int]]:
    return [(b, i) for b in range(B) for i in range(Lq)]


def gather_rows(t: torch.Tensor, rows: Sequence[Tuple[int, int]], layout: str) -> torch.Tensor:
    """Pick (b, i) rows: layout 'bihd' -> [n, H, D]; 'bhi' -> [n, H]; 'bgik' -> [n, Hkv, k]."""
    rb = torch.tensor([r[0] for r in rows], device=t.device)
    ri = torch.tensor([r[1] for r in rows], device=t.device)
    if layout == "bihd":
        return t[rb, ri]
    if layout == "bhi":
        return t[rb, :, ri]
    if layout == "bgik":
        return t[rb, :, ri]
    raise ValueError(layout)


def check_idx_against_oracle(idx_gpu: np.ndarray, idx_ref: np.ndarray, scores_ref: np.ndarray, rel=1e-3):
    """Rows [n, Hkv, k]; scores_ref [n, Hkv, Lk] are the oracle's probabilities.

    A GPU row may differ from the oracle's only by swapping keys whose oracle score is within `rel`
    (relative) of the row's k-th largest oracle score.  Returns the number of rows with a legal swap.
    """
    assert idx_gpu.shape == idx_ref.shape
    swapped = 0
    n, Hkv, k = idx_ref.shape
    for r in range(n):
        for g in range(Hkv):
            a, b = idx_gpu[r, g], idx_ref[r, g]
            if np.array_equal(a, b):
                continue
            sa, sb = a[a >= 0], b[b >= 0]
            assert len(sa) == len(sb), "row %d head %d: %d indices, oracle has %d" % (r, g, len(sa), len(sb))
            assert np.all(np.diff(sa) > 0), "row %d head %d: not strictly ascending" % (r, g)
            assert np.all(a[len(sa):] == -1)
            tau = scores_ref[r, g, sb].min()
            diff = np.setxor1d(sa, sb)
            sc = scores_ref[r, g, diff]
            assert np.all(np.abs(np.log(sc) - math.log(tau)) <= rel), \
                "row %d head %d: index swap outside the near-tie band: %s" % (r, g, diff[:8])
            swapped += 1
    return swapped


class BlockRun:
    """One FA layer + sparse layers on the GPU, with the oracle on chosen rows."""

    def __init__(self, inp, device="cuda"):
        self.inp = inp
        wl = inp.wl
        self.wl = wl
        self.dev = device
        self.q = inp.q_full.to(device)
        self.k = inp.k.to(device)
        self.v = inp.v.to(device)
        self.qs = [t.to(device) for t in inp.q_sparse]
        self.prob = hs2.Problem.from_tensors(self.q, self.k, wl.k_sel, wl.window)

    def run_full(self, want_scores=False, ws=None):
        self.O, self.LSE, self.idx, self.scores = hs2.hs2_full_attn_select(
            self.prob, self.q, self.k, self.v, want_scores=want_scores, ws=ws)
        torch.cuda.synchronize()
        return self

    def check_full(self, rows=None, check_scores=False):
        wl = self.wl
        rows = rows_all(wl.batch, wl.q_len) if rows is None else rows
        kh, vh = to_host(self.k), to_host(self.v)
        Oo, LSEo, idxo, sco = oracle.full_attn_select(to_host(self.q), kh, vh, wl.k_sel, wl.window, rows=rows,
                                                      want_scores=True)
        dt = wl.torch_dtype
        assert_output_close(gather_rows(self.O, rows, "bihd"), Oo, dt, "full attention O")
        lse = gather_rows(self.LSE, rows, "bhi").cpu().numpy().astype(np.float64)
        assert np.abs(lse - LSEo).max() <= TOL[dt]["lse"], "LSE max-abs %.3e" % np.abs(lse - LSEo).max()
        idx_gpu = gather_rows(self.idx, rows, "bgik").cpu().numpy()
        swaps = check_idx_against_oracle(idx_gpu, idxo, sco)
        if check_scores and self.scores is not None:
            sg = gather_rows(self.scores, rows, "bgik").cpu().numpy().astype(np.float64)
            vis = ~np.isneginf(sco)
            assert np.array_equal(np.isneginf(sg), ~vis), "visibility pattern of scores_dbg"
            err = np.abs(sg[vis] - np.log(sco[vis]))
            assert err.max() <= TOL[dt]["score"], "log-score max-abs %.3e" % err.max()
        return swaps

    def check_idx_bitexact_on_gpu_scores(self, rows=None):
        """The emitted indices are exactly the oracle's top-k of the fp32 scores the GPU reports."""
        wl = self.wl
        rows = rows_all(wl.batch, wl.q_len) if rows is None else rows
        sg = gather_rows(self.scores, rows, "bgik").cpu().numpy()          # [n, Hkv, Lk] fp32
        n, Hkv, Lk = sg.shape
        prob = oracle.Problem(to_host(self.q), to_host(self.k), wl.k_sel, wl.window)
        pos = np.repeat(np.array([prob.pos(b, i) for b, i in rows], dtype=np.int32), Hkv)
        kvl = np.repeat(np.array([prob.kvlen(b) for b, _ in rows], dtype=np.int32), Hkv)
        want = oracle.select(sg.reshape(n * Hkv, Lk), pos, kvl, wl.window, wl.k_sel).reshape(n, Hkv, wl.k_sel)
        got = gather_rows(self.idx, rows, "bgik").cpu().numpy()
        assert np.array_equal(got, want)

    def run_sparse(self, layer=0, decode=False, sink=None, want_lse=True, gate=None):
        fn = hs2.hs2_sparse_attn_decode if decode else hs2.hs2_sparse_attn_prefill
        out, lse = fn(self.prob, self.qs[layer], self.k, self.v, self.idx, sink=sink, want_lse=want_lse, gate=gate)
        torch.cuda.synchronize()
        return out, lse

    def check_sparse(self, out, lse, layer=0, rows=None, sink=None, gate=None):
        """Oracle sparse attention on the GPU's own indices (a legal tie swap must not pollute this check)."""
        wl = self.wl
        rows = rows_all(wl.batch, wl.q_len) if rows is None else rows
        idx_rows = gather_rows(self.idx, rows, "bgik").cpu().numpy()
        Oo, LSEo, _ = oracle.sparse_attn(to_host(self.qs[layer]), to_host(self.k), to_host(self.v), idx_rows,
                                         wl.window, rows=rows,
                                         sink=None if sink is None else sink.cpu().numpy().astype(np.float64),
                                         gate=None if gate is None else to_host(gate))
        dt = wl.torch_dtype
        assert_output_close(gather_rows(out, rows, "bihd"), Oo, dt, "sparse attention O")
        if lse is not None:
            l = gather_rows(lse, rows, "bhi").cpu().numpy().astype(np.float64)
            assert np.abs(l - LSEo).max() <= TOL[dt]["lse"], "sparse LSE max-abs %.3e" % np.abs(l - LSEo).max()

    def check_decode(self, out1, lse1, layer=0, sink=None, gate=None):
        """A decode call on the last query of every sequence against the oracle itself (not against the GPU's prefill
        row): sparse attention of row q_len-1 on the GPU's own indices, max-abs and mean-abs.  `out1` [B,1,Hq,D],
        `lse1` [B,Hq,1] or None, `gate` the prefill-shaped gate tensor or None."""
        wl = self.wl
        rows = [(b, wl.q_len - 1) for b in range(wl.batch)]
        idx_rows = gather_rows(self.idx, rows, "bgik").cpu().numpy()
        Oo, LSEo, _ = oracle.sparse_attn(to_host(self.qs[layer]), to_host(self.k), to_host(self.v), idx_rows,
                                         wl.window, rows=rows,
                                         sink=None if sink is None else sink.cpu().numpy().astype(np.float64),
                                         gate=None if gate is None else to_host(gate))
        dt = wl.torch_dtype
        assert_output_close(out1[:, 0], Oo, dt, "sparse decode O")
        if lse1 is not None:
            l = lse1[:, :, 0].cpu().numpy().astype(np.float64)
            assert np.abs(l - LSEo).max() <= TOL[dt]["lse"], "decode LSE max-abs %.3e" % np.abs(l - LSEo).max()
