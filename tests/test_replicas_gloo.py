"""The multi-GPU path has no collective in the data path; what there is - unit sharding and the
max-over-ranks timing reduction - is exercised here with two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_26368_b200.replicas import aggregate_throughput, shard_units


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
