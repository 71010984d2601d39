"""Host-side logic for running the path on several GPUs of one node.

The path has no exchange step: every (sequence, KV head) pair is an independent unit for the full
layer, the selection and the sparse layers (scores are aggregated only inside a KV-head group and
the indices are per KV head).  So ranks either run independent replicas of a workload (weak
scaling, what ``bench.py --gpus N`` does) or take disjoint slices of the units of one workload;
in both cases the only communication is the timing reduction below.  Works with any
``torch.distributed`` backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Tuple

import torch
import torch.distributed as dist


def shard_units(batch: int, n_kv_heads: int, rank: int, world: int) -> List[Tuple[int, int]]:
    """The (sequence, KV head) units rank `rank` owns: a contiguous, balanced slice of the B*Hkv units.

    Contiguous in (b, g) order so that a rank's slice of the cache, the queries of its head groups
    and its index rows are contiguous views; sizes differ by at most one unit.
    """
    n = batch * n_kv_heads
    base, extra = divmod(n, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return [(u // n_kv_heads, u % n_kv_heads) for u in range(lo, hi)]


def aggregate_throughput(units_local: float, ms_local: float, device="cpu") -> Tuple[float, float, float]:
    """Whole-job throughput from per-rank work and per-rank device time.

    Returns ``(units_per_second, total_units, max_ms)``: the units all ranks processed divided by the
    slowest rank's time.  Without an initialised process group it is the local ratio.
    """
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return units_local / (ms_local * 1e-3), units_local, ms_local
    t = torch.tensor([units_local], dtype=torch.float64, device=device)
    m = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    dist.all_reduce(m, op=dist.ReduceOp.MAX)
    return float(t.item()) / (float(m.item()) * 1e-3), float(t.item()), float(m.item())
