"""The decode entry point that brings its own scratch (hs2_sparse_attn_decode_static).

Some users of the library may not allocate device memory where they decode: a plugin that only
receives tensor pointers, a server whose memory pool owns the whole device, a loop that cannot take
the synchronisation an allocation implies.  For them the split-KV decode kernel keeps its partial
results in a fixed array inside the library.  This file checks, through the C ABI, that the call
gives what the ordinary decode entry point gives - on two calls in a row, because the second call
finds the first one's partials and tickets still sitting in the shared array - and that it refuses
problems beyond its stated limit.  It is collected last on purpose, and passes on its own too.
"""
import ctypes as C

import pytest
import torch

import numpy as np

import oracle
import paper_2609_26368_b200 as hs2
from paper_2609_26368_b200 import binding
from gen import make_inputs, scaled
from parity import TOL, assert_output_close, to_host

pytestmark = pytest.mark.gpu


def _case(batch, kv_len, k_sel, window, seed_shift, heads=(32, 4)):
    kw = dict(batch=batch, kv_len=kv_len, k_sel=k_sel, window=window, n_needles=8, n_q_heads=heads[0], n_kv_heads=heads[1])
    wl = scaled("cfg5", **kw)
    wl = scaled("cfg5", seed=wl.seed + seed_shift, **kw)
    inp = make_inputs(wl, "cuda")
    prob = hs2.Problem.from_tensors(inp.q_full, inp.k, wl.k_sel, wl.window)
    _, _, idx, _ = hs2.hs2_full_attn_select(prob, inp.q_full, inp.k, inp.v)
    return wl, inp, prob, idx


def test_static_scratch_decode_matches_the_workspace_decode_twice_in_a_row():
    assert torch.cuda.is_available()
    lib = hs2.load_library()
    # the third case has groups of 16 heads, which the kernel takes as two sub-groups of 8: 8 sequences x 4 KV heads are
    # 64 (sequence, sub-group) pairs, exactly the limit
    for call, (batch, kv_len, k_sel, window, heads) in enumerate([(8, 6000, 1024, 64, (32, 4)), (3, 2500, 700, 33, (32, 4)),
                                                                  (8, 3000, 512, 40, (64, 4))]):
        wl, inp, prob, idx = _case(batch, kv_len, k_sel, window, call, heads)
        sink = torch.linspace(-1.0, 1.0, heads[0], device="cuda")
        q = inp.q_sparse[0]
        ref, ref_lse = hs2.hs2_sparse_attn_decode(prob, q, inp.k, inp.v, idx, sink=sink, want_lse=True)
        out = torch.full_like(q, float("nan"))
        lse = torch.full_like(ref_lse, float("nan"))
        before = torch.cuda.memory_allocated()
        # straight through the C ABI: plain pointers, no workspace argument
        c = prob.c_struct(q, inp.k, out)
        st = lib.hs2_sparse_attn_decode_static(C.byref(c), q.data_ptr(), inp.k.data_ptr(), inp.v.data_ptr(),
                                               idx.data_ptr(), sink.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                               C.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert st == binding.HS2_OK, hs2.hs2_status_string(st)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert torch.isfinite(out.float()).all()
        # same kernel arithmetic, possibly another split count: the bf16 output tolerance of the parity tests
        assert (out.float() - ref.float()).abs().max().item() <= 2e-2
        assert (out.float() - ref.float()).abs().mean().item() <= 2e-3
        assert (lse - ref_lse).abs().max().item() <= 2e-3
        # and against the CPU oracle itself, on the same indices
        Oo, LSEo, _ = oracle.sparse_attn(to_host(q), to_host(inp.k), to_host(inp.v), idx[:, :, 0].cpu().numpy(), wl.window,
                                         sink=sink.cpu().numpy().astype(np.float64))
        assert_output_close(out[:, 0], Oo, torch.bfloat16, "static-scratch decode O")
        assert np.abs(lse[:, :, 0].cpu().numpy() - LSEo).max() <= TOL[torch.bfloat16]["lse"]
        # and once more through the Python binding, on the scratch the call above left behind
        out2, _ = hs2.hs2_sparse_attn_decode_static(prob, q, inp.k, inp.v, idx, sink=sink, out=torch.empty_like(q))
        torch.cuda.synchronize()
        assert torch.equal(out2, out)


def test_static_scratch_decode_refuses_what_does_not_fit():
    lib = hs2.load_library()
    one = C.c_void_p(256)            # never dereferenced: the size check comes before any launch
    big = hs2.Problem(batch=17, q_len=1, kv_len=4096, n_q_heads=32, n_kv_heads=4, head_dim=128, k_sel=256, window=16)
    st = lib.hs2_sparse_attn_decode_static(C.byref(big.c_struct()), one, one, one, one, None, one, None, None)
    assert st == binding.HS2_ERR_STATIC_SCRATCH
    assert "built-in" in hs2.hs2_status_string(st)
    # groups of 16 heads count twice: 9 sequences x 4 KV heads are 72 (sequence, sub-group) pairs
    g16 = hs2.Problem(batch=9, q_len=1, kv_len=4096, n_q_heads=64, n_kv_heads=4, head_dim=128, k_sel=256, window=16)
    st = lib.hs2_sparse_attn_decode_static(C.byref(g16.c_struct()), one, one, one, one, None, one, None, None)
    assert st == binding.HS2_ERR_STATIC_SCRATCH
    fp32 = hs2.Problem(batch=1, q_len=1, kv_len=512, n_q_heads=4, n_kv_heads=1, head_dim=64, k_sel=64, window=16,
                       dtype=torch.float32)
    st = lib.hs2_sparse_attn_decode_static(C.byref(fp32.c_struct()), one, one, one, one, None, one, None, None)
    assert st == binding.HS2_ERR_UNSUPPORTED
