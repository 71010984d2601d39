"""Host-side logic for running the path on several GPUs of one node.

The path has no exchange step: every (sequence, KV head) pair is an independent unit for the full
layer, the selection and the sparse layers (scores are aggregated only inside a KV-head group and
the indices are per KV head).  So ranks either run independent replicas of a workload (weak
scaling, what ``bench.py --gpus N`` does) or take disjoint slices of the units of one workload;
in both cases the only communication is the timing reduction below.  Works with any
``torch.distributed`` backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Sequence, Tuple

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


@dataclass(frozen=True)
class UnitSlice:
    """KV heads [g0, g1) of sequence b: a contiguous run of one rank's units."""
    b: int
    g0: int
    g1: int

    @property
    def n_kv_heads(self) -> int:
        return self.g1 - self.g0


def shard_slices(batch: int, n_kv_heads: int, rank: int, world: int) -> List[UnitSlice]:
    """The rank's units grouped into one slice per sequence it touches (each a sub-problem with batch 1)."""
    out: List[UnitSlice] = []
    for b, g in shard_units(batch, n_kv_heads, rank, world):
        if out and out[-1].b == b and out[-1].g1 == g:
            out[-1] = UnitSlice(b, out[-1].g0, g + 1)
        else:
            out.append(UnitSlice(b, g, g + 1))
    return out


def slice_inputs(sl: UnitSlice, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor):
    """Views (no copies) of Q ``[B, Lq, Hq, D]`` and K, V ``[B, Lk, Hkv, D]`` for one slice: the slice's KV heads and
    the query heads of their groups.  The views are strided; the library takes strides."""
    group = q.shape[2] // k.shape[2]
    return (q[sl.b:sl.b + 1, :, sl.g0 * group:sl.g1 * group], k[sl.b:sl.b + 1, :, sl.g0:sl.g1], v[sl.b:sl.b + 1, :, sl.g0:sl.g1])


def slice_problem(sl: UnitSlice, group: int, **problem_fields) -> Dict[str, int]:
    """Fields of the sub-problem one slice is: batch 1, its KV heads and their query heads; everything else
    (lengths, head_dim, k_sel, window, ...) as given."""
    return dict(problem_fields, batch=1, n_kv_heads=sl.n_kv_heads, n_q_heads=sl.n_kv_heads * group)


def reassemble(slices: Sequence[UnitSlice], parts: Sequence[Dict[str, torch.Tensor]], batch: int, n_kv_heads: int,
               group: int) -> Dict[str, torch.Tensor]:
    """Per-slice results back into the layouts of the whole problem.

    ``parts[n]`` holds any of ``O`` ``[1, Lq, heads, D]``, ``LSE`` ``[1, heads, Lq]``, ``idx`` ``[1, kv heads, Lq, k]``
    of slice ``slices[n]`` (all slices of all ranks, any order).  Every (sequence, KV head) must be covered once.
    """
    seen = set()
    out: Dict[str, torch.Tensor] = {}
    for sl, part in zip(slices, parts):
        for g in range(sl.g0, sl.g1):
            assert (sl.b, g) not in seen, "unit (%d, %d) appears twice" % (sl.b, g)
            seen.add((sl.b, g))
        for name, t in part.items():
            if name not in out:
                shape = list(t.shape)
                shape[0] = batch
                shape[2 if name == "O" else 1] = n_kv_heads * (1 if name == "idx" else group)
                out[name] = torch.empty(shape, dtype=t.dtype, device=t.device)
            if name == "O":
                out[name][sl.b, :, sl.g0 * group:sl.g1 * group] = t[0]
            elif name == "LSE":
                out[name][sl.b, sl.g0 * group:sl.g1 * group] = t[0]
            elif name == "idx":
                out[name][sl.b, sl.g0:sl.g1] = t[0]
            else:
                raise KeyError(name)
    assert len(seen) == batch * n_kv_heads, "units missing: %d of %d" % (len(seen), batch * n_kv_heads)
    return out


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
