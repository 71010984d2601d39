"""The multi-GPU path has no collective in the data path; what there is - unit sharding and the
max-over-ranks timing reduction - is exercised here with two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import numpy as np

import oracle
from gen import make_inputs, scaled
from paper_2609_26368_b200.replicas import (UnitSlice, aggregate_throughput, reassemble, shard_slices, shard_units,
                                            slice_inputs, slice_problem)


def test_shards_cover_every_unit_once_and_are_balanced():
    for batch, hkv in [(1, 4), (2, 4), (64, 4), (3, 1), (1, 1)]:
        for world in (1, 2, 3, 4, 8):
            parts = [shard_units(batch, hkv, r, world) for r in range(world)]
            flat = [u for p in parts for u in p]
            assert sorted(flat) == [(b, g) for b in range(batch) for g in range(hkv)]
            assert flat == sorted(flat)                                   # contiguous in (b, g) order
            sizes = [len(p) for p in parts]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    units = shard_units(2, 4, rank, world)
    ms = 10.0 if rank == 0 else 25.0                                       # rank 1 is the slow one
    val, total, mx = aggregate_throughput(float(len(units)) * 8192, ms)
    out[rank] = (val, total, mx, len(units))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_report_total_work_over_the_slowest_time():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0][3] + out[1][3] == 8
    for r in (0, 1):
        val, total, mx, _ = out[r]
        assert total == 8 * 8192 and mx == 25.0
        assert abs(val - 8 * 8192 / 25e-3) < 1e-6


def test_single_process_is_the_local_ratio():
    val, total, mx = aggregate_throughput(1000.0, 4.0)
    assert (val, total, mx) == (250000.0, 1000.0, 4.0)


# ---- a sharded problem end to end on the host side: units -> per-rank sub-problems and tensor slices -> results of the
# ---- slices put back into the whole problem's layouts.  The CPU oracle stands in for the GPU kernels as the thing that
# ---- computes a sub-problem (the library itself has no CPU path); what is under test is the sharding logic.

def _block_on(q, k, v, qs, k_sel, window):
    """One hybrid block on a (sub-)problem: full layer with selection, one sparse layer on its indices."""
    O, LSE, idx, _ = oracle.full_attn_select(q.contiguous(), k.contiguous(), v.contiguous(), k_sel, window)
    B, Lq, Hq, D = q.shape
    Hkv = k.shape[2]
    Os, _, _ = oracle.sparse_attn(qs.contiguous(), k.contiguous(), v.contiguous(), idx, window)
    return {"O": torch.from_numpy(Os.reshape(B, Lq, Hq, D)),
            "LSE": torch.from_numpy(LSE.reshape(B, Lq, Hq)).permute(0, 2, 1).contiguous(),
            "idx": torch.from_numpy(idx.reshape(B, Lq, Hkv, k_sel)).permute(0, 2, 1, 3).contiguous()}


def _sharded_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = scaled("cfg2", batch=3, q_len=40, kv_len=40, n_q_heads=6, n_kv_heads=3, head_dim=16, k_sel=6, window=4, n_needles=2)
    inp = make_inputs(wl)                                   # seeded: every rank draws the same bytes
    group = wl.n_q_heads // wl.n_kv_heads
    mine = shard_slices(wl.batch, wl.n_kv_heads, rank, world)
    parts = []
    for sl in mine:
        q, k, v = slice_inputs(sl, inp.q_full, inp.k, inp.v)
        qs, _, _ = slice_inputs(sl, inp.q_sparse[0], inp.k, inp.v)
        f = slice_problem(sl, group, q_len=wl.q_len, kv_len=wl.kv_len, head_dim=wl.head_dim, k_sel=wl.k_sel, window=wl.window)
        assert (f["batch"], f["n_kv_heads"], f["n_q_heads"]) == (1, k.shape[2], q.shape[2])
        assert q.data_ptr() >= inp.q_full.data_ptr() and not q.is_contiguous() or sl.n_kv_heads == wl.n_kv_heads   # a view
        parts.append(_block_on(q, k, v, qs, wl.k_sel, wl.window))
    gathered = [None] * world
    dist.all_gather_object(gathered, (mine, parts))          # test plumbing; the data path itself exchanges nothing
    slices = [s for r in gathered for s in r[0]]
    allparts = [p for r in gathered for p in r[1]]
    whole = reassemble(slices, allparts, wl.batch, wl.n_kv_heads, group)
    ref = _block_on(inp.q_full, inp.k, inp.v, inp.q_sparse[0], wl.k_sel, wl.window)
    out[rank] = (len(mine), all(torch.equal(whole[n], ref[n]) for n in ("O", "LSE", "idx")),
                 tuple(whole["idx"].shape), tuple(whole["O"].shape))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_run_a_sharded_block_and_reassemble_it():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_sharded_worker, args=(2, port, out), nprocs=2, join=True)
    for r in (0, 1):
        n_slices, same, idx_shape, o_shape = out[r]
        assert same, "reassembled results differ from the unsharded block on rank %d" % r
        assert idx_shape == (3, 3, 40, 6) and o_shape == (3, 40, 6, 16)
    assert out[0][0] + out[1][0] == 4            # 9 units as 5 + 4: slices (0, 0-3), (1, 0-2) | (1, 2-3), (2, 0-3)


def test_slices_follow_the_units():
    assert shard_slices(2, 4, 0, 3) == [UnitSlice(0, 0, 3)]
    assert shard_slices(2, 4, 1, 3) == [UnitSlice(0, 3, 4), UnitSlice(1, 0, 2)]
    assert shard_slices(2, 4, 2, 3) == [UnitSlice(1, 2, 4)]
    assert shard_slices(1, 1, 1, 2) == []
