"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the whole block
runs on the GPU, the oracle checks sampled query rows one by one (budget edges + seeded uniform rows,
all heads), and properties that hold for every row are checked on the full outputs."""
import numpy as np
import pytest
import torch

import paper_2609_26368_b200 as hs2
from gen import CONFIGS, make_inputs, sample_rows
from gen.workloads import NATIVE
from parity import BlockRun

pytestmark = pytest.mark.gpu


def _index_properties(run, stride=1):
    """Every idx row: ascending, unique, in range, outside the window, right count, -1 padded."""
    wl = run.wl
    idx = run.idx[:, :, ::stride]                                  # [B, Hkv, n, k]
    B, Hkv, n, k = idx.shape
    q0 = wl.kv_len - wl.q_len
    pos = (torch.arange(0, wl.q_len, stride, device=idx.device) + q0).view(1, 1, n, 1)
    valid = idx >= 0
    want = torch.clamp(pos - wl.window + 1, min=0).clamp(max=k).view(1, 1, n)
    assert torch.equal(valid.sum(-1), want.expand(B, Hkv, n))
    slot = torch.arange(k, device=idx.device).view(1, 1, 1, k)
    assert bool((valid == (slot < want.unsqueeze(-1))).all())      # padding only at the end
    assert bool(((idx <= pos - wl.window) | ~valid).all())         # never inside the window / the future
    inc = (idx[..., 1:] > idx[..., :-1]) | ~valid[..., 1:]
    assert bool(inc.all())                                         # strictly ascending => unique


def _run_block(name, n_rows, layers=None, wl=None):
    if wl is None:
        wl = CONFIGS[name] if name in CONFIGS else NATIVE[name]
    inp = make_inputs(wl, "cuda")
    run = BlockRun(inp).run_full()
    rows = [(b, i) for b in range(wl.batch) for i in sample_rows(wl, n_rows)]
    swaps = run.check_full(rows=rows)
    _index_properties(run, stride=max(1, wl.q_len // 4096))
    for layer in (range(len(run.qs)) if layers is None else layers):
        fn_decode = wl.q_len == 1
        out, lse = run.run_sparse(layer, decode=fn_decode)
        assert bool(torch.isfinite(out.float()).all())
        run.check_sparse(out, lse, layer, rows=rows)
    return swaps


def test_cfg2_full_size_sampled():
    _run_block("cfg2", 256)


def test_cfg3_full_size_sampled():
    _run_block("cfg3", 64)


def test_cfg4_full_size_sampled():
    _run_block("cfg4", 64)


def test_cfg5_decode_full_size_every_sequence():
    _run_block("cfg5", 1)


def test_native8k_full_size_sampled():
    """The paper's own attention shape (64 query heads on one KV head, head_dim 256) as bench.py times it: every kernel
    of the block on tcgen05."""
    _run_block("native8k", 64)


def test_native_decode_full_size_every_sequence():
    """Decode at the paper's shape, batch 64 on a 64K-token cache: the splits of a sequence merge inside a cluster."""
    _run_block("native_decode", 1, layers=[0])


def test_native_shape_at_a_32k_context_sampled():
    """The paper's shape at the longer context bench.py also times: score strips of 32768 keys, rows for the cluster
    top-k's smaller sibling, 32768 work items of the tensor-core gather kernel."""
    import dataclasses
    wl = dataclasses.replace(NATIVE["native8k"], q_len=32768, kv_len=32768, name="native32k")
    _run_block("native32k", 16, layers=[0], wl=wl)
