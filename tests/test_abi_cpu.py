"""CPU-only checks of the C-ABI library: it loads, exports what include/hs2.h declares, sizes its
workspace on the host and rejects bad arguments before touching a GPU."""
import ctypes as C
import os
import re

import pytest
import torch

import paper_2609_26368_b200 as hs2
from paper_2609_26368_b200 import binding
from paper_2609_26368_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build()
    return hs2.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "hs2.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(hs2_[a-z0-9_]+)\s*\(", header)))
    assert set(binding.EXPORTS) == set(declared)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    texts = [hs2.hs2_status_string(s) for s in range(6)]
    assert texts[0] == "ok" and len(set(texts)) == 6
    assert hs2.hs2_status_string(99) == "unknown status"


def _prob(**kw):
    d = dict(batch=1, q_len=64, kv_len=64, n_q_heads=4, n_kv_heads=1, head_dim=64, k_sel=8, window=4,
             dtype=torch.float32)
    d.update(kw)
    return hs2.Problem(**d)


def test_workspace_sizes_are_host_side(lib):
    p = _prob()
    assert hs2.hs2_workspace_bytes(p, binding.HS2_OP_FULL_ATTN_SELECT) == 64 * 64 * 4
    assert hs2.hs2_workspace_bytes(p, binding.HS2_OP_TOPK_SELECT) == 0
    assert hs2.hs2_workspace_bytes(p, binding.HS2_OP_SPARSE_ATTN_PREFILL) == 0
    big = _prob(q_len=131072, kv_len=131072, n_q_heads=32, n_kv_heads=4, head_dim=128, dtype=torch.bfloat16)
    n = hs2.hs2_workspace_bytes(big, binding.HS2_OP_FULL_ATTN_SELECT)                   # capped, whatever the path
    assert (1 << 30) <= n <= (1 << 30) + (1 << 20)
    assert hs2.hs2_workspace_bytes(_prob(n_q_heads=3, n_kv_heads=2), binding.HS2_OP_FULL_ATTN_SELECT) == 0


@pytest.mark.parametrize("bad", [
    dict(batch=0), dict(q_len=0), dict(kv_len=-1), dict(n_q_heads=3, n_kv_heads=2), dict(head_dim=0),
    dict(k_sel=-1), dict(window=-2), dict(k_sel=0, window=0), dict(softmax_scale=float("nan")),
    dict(softmax_scale=-1.0),
])
def test_invalid_problems_are_rejected_without_a_launch(lib, bad):
    c = _prob(**bad).c_struct()
    one = C.c_void_p(256)          # never dereferenced: validation fails first
    st = lib.hs2_sparse_attn_prefill(C.byref(c), one, one, one, one, None, one, None, None, 0, None)
    assert st == binding.HS2_ERR_INVALID_ARG
    st = lib.hs2_full_attn_select(C.byref(c), one, one, one, one, one, one, None, one, 1 << 20, None)
    assert st == binding.HS2_ERR_INVALID_ARG


def test_unsupported_and_null_and_workspace_errors(lib):
    one = C.c_void_p(256)
    c = _prob(head_dim=512).c_struct()
    assert lib.hs2_sparse_attn_prefill(C.byref(c), one, one, one, one, None, one, None, None, 0, None) == \
        binding.HS2_ERR_UNSUPPORTED
    c = _prob().c_struct()
    assert lib.hs2_sparse_attn_prefill(C.byref(c), None, one, one, one, None, one, None, None, 0, None) == \
        binding.HS2_ERR_INVALID_ARG
    assert lib.hs2_sparse_attn_prefill(C.byref(c), one, one, one, None, None, one, None, None, 0, None) == \
        binding.HS2_ERR_INVALID_ARG                                  # idx required when k_sel > 0
    assert lib.hs2_full_attn_select(C.byref(c), one, one, one, one, None, one, None, one, 1 << 20, None) == \
        binding.HS2_ERR_INVALID_ARG                                  # LSE required
    assert lib.hs2_full_attn_select(C.byref(c), one, one, one, one, one, one, None, one, 16, None) == \
        binding.HS2_ERR_WORKSPACE_TOO_SMALL
    assert lib.hs2_full_attn_select(C.byref(c), one, one, one, one, one, one, None, C.c_void_p(260), 1 << 20, None) == \
        binding.HS2_ERR_WORKSPACE_TOO_SMALL                          # misaligned
    c2 = _prob(q_len=2).c_struct()
    assert lib.hs2_sparse_attn_decode(C.byref(c2), one, one, one, one, None, one, None, None, 0, None) == \
        binding.HS2_ERR_INVALID_ARG                                  # decode wants q_len == 1
    c3 = _prob().c_struct()
    c3.q_stride = (C.c_int64 * 3)(64 * 4 * 64, 4 * 64, 32)           # head stride below head_dim
    assert lib.hs2_sparse_attn_prefill(C.byref(c3), one, one, one, one, None, one, None, None, 0, None) == \
        binding.HS2_ERR_INVALID_ARG


def test_fp8_record_layout_argument_checks(lib):
    one = C.c_void_p(256)
    c = _prob(head_dim=128, dtype=torch.bfloat16).c_struct()
    c.kv_scale_stride = (C.c_int64 * 3)(64 * 72, 72, 0)              # scales of two heads on top of each other
    assert lib.hs2_sparse_attn_prefill_fp8kv(C.byref(c), one, one, one, one, one, one, None, one, None, None) == \
        binding.HS2_ERR_INVALID_ARG
    c.kv_scale_stride = (C.c_int64 * 3)(-1, 72, 72)
    assert lib.hs2_sparse_attn_prefill_fp8kv(C.byref(c), one, one, one, one, one, one, None, one, None, None) == \
        binding.HS2_ERR_INVALID_ARG
    # the producer: a group stride below a group's 128 bytes, a missing scale pointer, rows that cannot hold their groups
    assert lib.hs2_kv_project_fp8_records(256, 64, 256, one, 64, one, 64, one, 576, 64, one, 144, 72, None) == \
        binding.HS2_ERR_INVALID_ARG
    assert lib.hs2_kv_project_fp8_records(256, 64, 256, one, 64, one, 64, one, 576, 288, None, 144, 72, None) == \
        binding.HS2_ERR_INVALID_ARG
    assert lib.hs2_kv_project_fp8_records(256, 64, 256, one, 64, one, 64, one, 288, 288, one, 144, 72, None) == \
        binding.HS2_ERR_UNSUPPORTED
    assert lib.hs2_kv_project_fp8_records(0, 64, 256, one, 64, one, 64, one, 576, 288, one, 144, 72, None) == binding.HS2_OK


def test_gather_probe_argument_checks(lib):
    one = C.c_void_p(256)
    bf = _prob(head_dim=128, dtype=torch.bfloat16).c_struct()
    assert lib.hs2_probe_gather(C.byref(bf), one, one, one, 0, None, None) == binding.HS2_ERR_INVALID_ARG   # no sink word
    assert lib.hs2_probe_gather(C.byref(bf), one, one, one, 2, one, None) == binding.HS2_ERR_INVALID_ARG    # mode 0 or 1
    assert lib.hs2_probe_gather(C.byref(bf), one, one, None, 0, one, None) == binding.HS2_ERR_INVALID_ARG   # idx needed
    assert lib.hs2_probe_gather(C.byref(_prob().c_struct()), one, one, one, 0, one, None) == binding.HS2_ERR_UNSUPPORTED


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU behaviour")
def test_no_gpu_means_an_error_not_a_fallback(lib):
    one = C.c_void_p(256)
    c = _prob().c_struct()
    st = lib.hs2_sparse_attn_prefill(C.byref(c), one, one, one, one, None, one, None, None, 0, None)
    assert st == binding.HS2_ERR_CUDA and lib.hs2_last_cuda_error() != 0
