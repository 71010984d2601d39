#!/usr/bin/env python
"""Benchmark of the hybrid sparse-attention hot path on B200.

One *step* is one pass of the whole path over one batch of synthetic input of the chosen
workload (default: the largest single-GPU prefill configuration, "cfg4": L=131072, one full layer and
three sparse layers; the two smaller prefill configurations are timed briefly as side sections):

    hs2_full_attn_select          full-attention layer + token-level top-k indices
    hs2_sparse_attn_prefill  x n  the sparse layers that reuse the cache and the indices
    hs2_full_attn_select (Lq=1) + hs2_sparse_attn_decode   one decode step on the same cache

The JSON line's `value` is tokens/s of that step with inputs resident in HBM; `roofline` describes
the sparse-prefill kernel: gathered K/V bytes per launch over its CUDA-event duration against the
measured HBM peak (`frac`, which exceeds 1 when a KV head's cache is L2 resident) and against a gather
ceiling measured in the same run (`frac_l2`: the same rows fetched by a kernel that does nothing else);
`decode_64k` times the split-KV decode kernel on the 64K-context configuration;
`e2e` repeats the step with pinned host inputs/outputs copied inside the timed region;
`cpu_baseline` is the CPU oracle on a bounded sample of the same workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload cfg4]

`--gpus N` with N > 1 started as a plain process re-executes itself under torch.distributed.run with
one rank per GPU (independent replicas of the workload; NCCL only for the barrier and the reduction
of the timings).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# torch.distributed.run sets OMP_NUM_THREADS=1 for its ranks; the CPU-oracle arm runs on rank 0 alone and is meant to use
# the machine's host cores, so it takes them back before any OpenMP runtime reads the variable
if "reference" in sys.argv and os.environ.get("RANK", "0") == "0" and os.environ.get("OMP_NUM_THREADS") == "1" \
        and "TORCHELASTIC_RUN_ID" in os.environ:
    os.environ["OMP_NUM_THREADS"] = str(os.cpu_count() or 1)

import torch  # noqa: E402

from gen import CONFIGS, make_inputs, sample_rows  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum of one k_sparse_prefill launch (bytes): RECORDED from ncu captures,
# not measured by this program.  Each entry names the summary under profiles/ that holds the capture's command.
NCU_DRAM_TRAFFIC = {
    "cfg2": (268.1e6, "profiles/block_step_cfg2.md"),
    "cfg4": (15.659e9, "profiles/sparse_prefill_dram_traffic.md"),
    "cfg4_len32768": (2.750e9, "profiles/sparse_prefill_dram_traffic.md"),
}

METRIC = "sparse-attn prefill tokens/s (hybrid block step: full-attn+select, sparse layers, decode step)"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------ workload arithmetic (host side)

def attended_tokens(wl) -> float:
    """Sum over queries of |S| = min(p+1, w) + min(k, max(0, p+1-w)) for one (sequence, KV head)."""
    q0 = wl.kv_len - wl.q_len
    total = 0
    for i in range(wl.q_len):
        p = q0 + i
        total += min(p + 1, wl.window) + min(wl.k_sel, max(0, p + 1 - wl.window))
    return float(total)


def gathered_kv_bytes(wl) -> float:
    """Algorithmic bytes of one sparse layer: every attended K row and V row once per (query, KV head)."""
    elt = 4 if wl.dtype == "f32" else 2
    return attended_tokens(wl) * wl.batch * wl.n_kv_heads * 2 * wl.head_dim * elt


def full_attn_flops(wl) -> float:
    """4 * D flops per (query head, visible key) pair: QK^T and PV, causal."""
    q0 = wl.kv_len - wl.q_len
    pairs = sum(min(q0 + i + 1, wl.kv_len) for i in range(wl.q_len))
    return 4.0 * wl.head_dim * wl.batch * wl.n_q_heads * pairs


def sparse_attn_flops(wl) -> float:
    """4 * D flops per (query head, attended key) pair of one sparse layer."""
    return 4.0 * wl.head_dim * attended_tokens(wl) * wl.batch * wl.n_q_heads


def oracle_row_flops(wl) -> float:
    """Average multiply-adds x 2 of one oracle query row (all heads): full attention + the sparse layers."""
    return full_attn_flops(wl) / (wl.batch * wl.q_len) + wl.n_sparse_layers * sparse_attn_flops(wl) / (wl.batch * wl.q_len)


def tensor_peak_for(ms: float, peaks):
    """Which measured bf16 peak a tensor-core kernel of this duration is held against: the burst figure for a kernel
    of a few milliseconds (it finishes before the power cap bites), the sustained one for longer kernels."""
    if ms < 5.0:
        return peaks["bf16_tflops"], "burst"
    return peaks["bf16_tflops_sustained"], "sustained"


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.lines, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        rows = [l for (t, l) in self.lines if (t0 is None or t >= t0 - 0.2) and (t1 is None or t <= t1 + 0.2)]
        rows = rows or [l for _, l in self.lines]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------ the step

class Block:
    """Device tensors and pre-allocated outputs of one hybrid block; `step()` enqueues the whole path."""

    def __init__(self, wl, device, rank=0):
        import paper_2609_26368_b200 as hs2
        from paper_2609_26368_b200 import binding
        self.hs2, self.wl, self.dev = hs2, wl, device
        from dataclasses import replace
        inp = make_inputs(replace(wl, seed=wl.seed + 1000 * rank), device)
        self.q_full, self.k, self.v, self.q_sparse = inp.q_full, inp.k, inp.v, inp.q_sparse
        self.prob = hs2.Problem.from_tensors(self.q_full, self.k, wl.k_sel, wl.window)
        B, Lq, Hq, D = self.q_full.shape
        Hkv = wl.n_kv_heads
        self.O_full = torch.empty_like(self.q_full)
        self.LSE = torch.empty(B, Hq, Lq, dtype=torch.float32, device=device)
        self.idx = torch.empty(B, Hkv, Lq, wl.k_sel, dtype=torch.int32, device=device)
        self.O_sparse = [torch.empty_like(self.q_full) for _ in self.q_sparse]
        self.ws_full = torch.empty(max(256, hs2.hs2_workspace_bytes(self.prob, binding.HS2_OP_FULL_ATTN_SELECT)),
                                   dtype=torch.uint8, device=device)
        self.ws_none = torch.empty(256, dtype=torch.uint8, device=device)
        # decode step on the same cache: the last token of every sequence
        self.with_decode = Lq > 1
        if self.with_decode:
            self.q1_full = self.q_full[:, -1:].contiguous()
            self.q1_sparse = [q[:, -1:].contiguous() for q in self.q_sparse]
            self.prob1 = hs2.Problem.from_tensors(self.q1_full, self.k, wl.k_sel, wl.window)
            self.O1_full = torch.empty_like(self.q1_full)
            self.LSE1 = torch.empty(B, Hq, 1, dtype=torch.float32, device=device)
            self.idx1 = torch.empty(B, Hkv, 1, wl.k_sel, dtype=torch.int32, device=device)
            self.O1_sparse = [torch.empty_like(self.q1_full) for _ in self.q_sparse]
            self.ws_full1 = torch.empty(max(256, hs2.hs2_workspace_bytes(self.prob1, binding.HS2_OP_FULL_ATTN_SELECT)),
                                        dtype=torch.uint8, device=device)
            self.ws_dec = torch.empty(max(256, hs2.hs2_workspace_bytes(self.prob1, binding.HS2_OP_SPARSE_ATTN_DECODE)),
                                      dtype=torch.uint8, device=device)
        self.kernel_ms = {}     # name -> list of (start_event, end_event)

    def _timed(self, name, fn, timing):
        if not timing:
            fn()
            return
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        self.kernel_ms.setdefault(name, []).append((a, b))

    def step(self, timing=False):
        hs2 = self.hs2
        self._timed("full_attn_select", lambda: hs2.hs2_full_attn_select(
            self.prob, self.q_full, self.k, self.v, out=self.O_full, lse=self.LSE, idx=self.idx, ws=self.ws_full), timing)
        for l, q in enumerate(self.q_sparse):
            self._timed("sparse_attn_prefill", lambda: hs2.hs2_sparse_attn_prefill(
                self.prob, q, self.k, self.v, self.idx, out=self.O_sparse[l], ws=self.ws_none), timing)
        if self.with_decode:
            self._timed("decode_full_attn_select", lambda: hs2.hs2_full_attn_select(
                self.prob1, self.q1_full, self.k, self.v, out=self.O1_full, lse=self.LSE1, idx=self.idx1,
                ws=self.ws_full1), timing)
            for l, q in enumerate(self.q1_sparse):
                self._timed("sparse_attn_decode", lambda: hs2.hs2_sparse_attn_decode(
                    self.prob1, q, self.k, self.v, self.idx1, out=self.O1_sparse[l], ws=self.ws_dec), timing)

    def gather_ceiling_ms(self, reps=3):
        """Duration of the bare row gather of one sparse layer (hs2_probe_gather: the same rows in the same order,
        nothing else), best of the two load modes, median of `reps` after one warm-up each.  Needs self.idx."""
        best = None
        self.probe_ms_by_mode = {}
        word = torch.zeros(1, dtype=torch.int32, device=self.dev)
        for mode in (0, 1):
            self.hs2.hs2_probe_gather(self.prob, self.k, self.v, self.idx, mode=mode, sink_word=word)
            ts = []
            for _ in range(reps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                self.hs2.hs2_probe_gather(self.prob, self.k, self.v, self.idx, mode=mode, sink_word=word)
                b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            t = statistics.median(ts)
            self.probe_ms_by_mode[mode] = t
            if best is None or t < best[0]:
                best = (t, mode)
        return best

    def kernel_means(self):
        return {k: sum(a.elapsed_time(b) for a, b in v) / len(v) for k, v in self.kernel_ms.items()}

    def input_bytes(self):
        ts = [self.q_full, self.k, self.v] + self.q_sparse
        return sum(t.numel() * t.element_size() for t in ts)

    def output_tensors(self):
        return [self.O_full] + self.O_sparse


def respawn_under_torchrun(n_gpus):
    """`bench.py --gpus N` started as a plain process: run the same command line as N ranks, one per GPU."""
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n_gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.stdout.flush()
    os.execv(sys.executable, cmd)


def dist_setup(n_gpus):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


def max_over_ranks(x: float, world, device):
    """Slowest rank's device time (the data path itself has no collective)."""
    from paper_2609_26368_b200.replicas import aggregate_throughput
    return aggregate_throughput(0.0, x, device)[2]


def time_steps(block, steps, warmup, world, timing=True, before=None, after=None):
    """W untimed steps, then exactly K steps between barrier+synchronize; device time in ms."""
    for _ in range(warmup):
        if before:
            before()
        block.step()
        if after:
            after()
    block.kernel_ms = {}
    barrier(world)
    block.launches0 = block.hs2.hs2_launch_count()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        if before:
            before()
        block.step(timing=timing)
        if after:
            after()
    b.record()
    block.launches = block.hs2.hs2_launch_count() - block.launches0
    torch.cuda.synchronize()
    barrier(world)
    return a.elapsed_time(b)


def time_e2e(wl, device, rank, block0, steps, world):
    """The same step fed from pinned host memory: every step copies its inputs host->device and its
    outputs device->host inside the timed region.  Two device buffer sets and three streams let the
    copies of neighbouring steps overlap the kernels (the user-level double buffering any server does)."""
    blocks = [block0, Block(wl, device, rank)]
    host_in = [t.cpu().pin_memory() for t in [block0.q_full, block0.k, block0.v] + block0.q_sparse]
    host_out = [[torch.empty(t.shape, dtype=t.dtype, device="cpu").pin_memory() for t in b.output_tensors()] for b in blocks]
    s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in blocks]      # inputs of buffer set landed
    ev_run = [torch.cuda.Event() for _ in blocks]     # kernels of buffer set finished
    ev_out = [torch.cuda.Event() for _ in blocks]     # outputs of buffer set copied back
    # the kernels of one step replay from a CUDA graph per buffer set: under concurrent copies the launches of the
    # short decode kernels otherwise queue behind the copy traffic
    graphs = []
    for b in blocks:
        with torch.cuda.stream(s_run):
            b.step()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s_run):
            b.step()
        graphs.append(g)
    torch.cuda.synchronize()

    def run(n):
        for it in range(n):
            b = blocks[it & 1]
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_run[it & 1])           # the set's previous kernels no longer read the inputs
                for d, h in zip([b.q_full, b.k, b.v] + b.q_sparse, host_in):
                    d.copy_(h, non_blocking=True)
                ev_in[it & 1].record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(ev_in[it & 1])
                s_run.wait_event(ev_out[it & 1])          # the set's previous outputs have left the device
                graphs[it & 1].replay()
                ev_run[it & 1].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_run[it & 1])
                for h, d in zip(host_out[it & 1], b.output_tensors()):
                    h.copy_(d, non_blocking=True)
                ev_out[it & 1].record(s_out)
    run(2)
    barrier(world)
    a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()                                         # default stream: everything before is done (synchronised)
    for st in (s_in, s_run, s_out):
        st.wait_event(a)
    run(steps)
    cur = torch.cuda.current_stream()
    for st in (s_in, s_run, s_out):
        done = torch.cuda.Event()
        done.record(st)
        cur.wait_event(done)
    e.record()
    torch.cuda.synchronize()
    barrier(world)
    del blocks[1]
    return a.elapsed_time(e)


# ------------------------------------------------------------------ decode at 64K context (cfg5)

def bench_decode_64k(device, peaks, reps=5, burst=40, ctx=65536, batch=0):
    """Split-KV sparse decode on the 64K-context configuration; indices from the full layer's scores.

    The cache (8.6 GB) is far above L2; consecutive launches rotate over four query/index sets so
    that no launch re-reads rows that the previous one left in L2.
    """
    import paper_2609_26368_b200 as hs2
    from paper_2609_26368_b200 import binding
    from dataclasses import replace
    wl = replace(CONFIGS["cfg5"], kv_len=ctx)
    if batch > 0:
        wl = replace(wl, batch=batch)
    inp = make_inputs(wl, device)
    k, v = inp.k, inp.v
    B, _, Hq, D = inp.q_full.shape
    prob = hs2.Problem.from_tensors(inp.q_full, k, wl.k_sel, wl.window)
    ws_full = torch.empty(max(256, hs2.hs2_workspace_bytes(prob, binding.HS2_OP_FULL_ATTN_SELECT)), dtype=torch.uint8, device=device)
    ws_dec = torch.empty(max(256, hs2.hs2_workspace_bytes(prob, binding.HS2_OP_SPARSE_ATTN_DECODE)), dtype=torch.uint8, device=device)
    nset = 4
    qfs = [inp.q_full] + [torch.randn_like(inp.q_full) for _ in range(nset - 1)]
    qss = [torch.randn_like(inp.q_full) for _ in range(nset)]
    idxs, t_full = [], []
    for s in range(nset):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        _, _, idx, _ = hs2.hs2_full_attn_select(prob, qfs[s], k, v, ws=ws_full)
        b.record()
        torch.cuda.synchronize()
        t_full.append(a.elapsed_time(b))
        idxs.append(idx)
    out = torch.empty_like(inp.q_full)

    def run(n):
        for it in range(n):
            hs2.hs2_sparse_attn_decode(prob, qss[it % nset], k, v, idxs[it % nset], out=out, ws=ws_dec)
    run(8)
    torch.cuda.synchronize()
    per = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        run(burst)
        b.record()
        torch.cuda.synchronize()
        per.append(a.elapsed_time(b) / burst)
    us = statistics.median(per) * 1e3
    gb = gathered_kv_bytes(wl)
    ach = gb / (us * 1e-6) / 1e9
    # the same step on an e4m3 cache (codes + one fp32 scale per (token, KV head)): 264 B per attended token
    from gen.workloads import quantize_kv_e4m3
    k8, ksc = quantize_kv_e4m3(k)
    v8, vsc = quantize_kv_e4m3(v)
    prob8 = hs2.Problem.from_tensors(inp.q_full, k8, wl.k_sel, wl.window)

    def run8(n):
        for it in range(n):
            hs2.hs2_sparse_attn_decode_fp8kv(prob8, qss[it % nset], k8, v8, ksc, vsc, idxs[it % nset], out=out)
    run8(8)
    torch.cuda.synchronize()
    per8 = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        run8(burst)
        b.record()
        torch.cuda.synchronize()
        per8.append(a.elapsed_time(b) / burst)
    us8 = statistics.median(per8) * 1e3
    gb8 = gb / 512.0 * 264.0
    # the full layer's decode step on the same cache (a sweep over all of it: codes + scales of K and V)
    ws8 = torch.empty(max(256, hs2.hs2_workspace_bytes(prob8, binding.HS2_OP_FULL_ATTN_SELECT_FP8KV)), dtype=torch.uint8, device=device)
    t_full8 = []
    for s in range(nset):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        hs2.hs2_full_attn_select_fp8kv(prob8, qfs[s], k8, v8, ksc, vsc, ws=ws8)
        b.record()
        torch.cuda.synchronize()
        t_full8.append(a.elapsed_time(b))
    sweep8 = (k8.numel() + v8.numel() + 4 * (ksc.numel() + vsc.numel())) / 1e9
    # the same cache as records [K codes | V codes | K scale | V scale | 24 spare bytes] per (token, KV head), which the
    # library reads through kv_stride and kv_scale_stride: one DRAM page per attended token and head instead of four
    Bc, Lc, Hc, Dc = k8.shape
    rec = torch.zeros(Bc, Lc, Hc, 2 * Dc + 32, dtype=torch.uint8, device=device)
    rec[..., :Dc].copy_(k8)
    rec[..., Dc:2 * Dc].copy_(v8)
    recf = rec.view(torch.float32)
    recf[..., 2 * Dc // 4].copy_(ksc)
    recf[..., 2 * Dc // 4 + 1].copy_(vsc)
    rk, rv, rks, rvs = rec[..., :Dc], rec[..., Dc:2 * Dc], recf[..., 2 * Dc // 4], recf[..., 2 * Dc // 4 + 1]
    del k8, v8, ksc, vsc

    def run8r(n):
        for it in range(n):
            hs2.hs2_sparse_attn_decode_fp8kv(prob8, qss[it % nset], rk, rv, rks, rvs, idxs[it % nset], out=out)
    run8r(8)
    torch.cuda.synchronize()
    per8r = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        run8r(burst)
        b.record()
        torch.cuda.synchronize()
        per8r.append(a.elapsed_time(b) / burst)
    us8r = statistics.median(per8r) * 1e3
    t_full8r = []
    for s in range(nset):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        hs2.hs2_full_attn_select_fp8kv(prob8, qfs[s], rk, rv, rks, rvs, ws=ws8)
        b.record()
        torch.cuda.synchronize()
        t_full8r.append(a.elapsed_time(b))
    fp8 = {"sparse_decode_us_per_step": round(us8, 2), "gathered_kv_bytes": gb8,
           "achieved_gbs": round(gb8 / (us8 * 1e-6) / 1e9, 1), "frac": round(gb8 / (us8 * 1e-6) / 1e9 / peaks["hbm_gbs"], 4),
           "full_attn_select_decode_ms": round(min(t_full8[1:]), 3), "cache_sweep_gb": round(sweep8, 2),
           "cache_sweep_ms_at_hbm_peak": round(sweep8 / peaks["hbm_gbs"] * 1e3, 3),
           "records_288B": {"sparse_decode_us_per_step": round(us8r, 2),
                            "frac": round(gb8 / (us8r * 1e-6) / 1e9 / peaks["hbm_gbs"], 4),
                            "full_attn_select_decode_ms": round(min(t_full8r[1:]), 3),
                            "layout": "K codes, V codes and both scales of a (token, KV head) in one 288-byte record (whole 32-byte sectors; 272-byte records: 40.7 us)"}}
    return {"workload": "cfg5: B=%d, ctx %d, 32q/4kv, D=128, bf16, k=2048, w=128" % (wl.batch, ctx), "fp8_kv_cache": fp8,
            "sparse_decode_us_per_step": round(us, 2), "gathered_kv_bytes": gb,
            "achieved_gbs": round(ach, 1), "peak_gbs": peaks["hbm_gbs"], "frac": round(ach / peaks["hbm_gbs"], 4),
            "full_attn_select_decode_ms": round(min(t_full[1:]), 3), "launches_back_to_back": burst,
            "l2": "%.1f GB cache, 4 rotating query/index sets (1.1 GB of gathered rows) > L2" % (2 * k.numel() * 2 / 1e9)}


def bench_native(device, peaks, reps=5):
    """The paper's own attention shape (Table 1: 64 query heads on one KV head, head_dim 256, 1024 selected + 128
    window tokens): full layer with selection and sparse prefill at 8K, sparse decode at batch 64 and a 64K cache.
    Reported beside the benchmark configurations; every kernel on this path is a tcgen05 kernel."""
    import paper_2609_26368_b200 as hs2
    from paper_2609_26368_b200 import binding
    from gen.workloads import NATIVE

    def med(fn, n=reps, warm=2):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(n):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)

    out = {}
    wl = NATIVE["native8k"]
    inp = make_inputs(wl, device)
    q, k, v = inp.q_full, inp.k, inp.v
    prob = hs2.Problem.from_tensors(q, k, wl.k_sel, wl.window)
    ws = torch.empty(max(256, hs2.hs2_workspace_bytes(prob, binding.HS2_OP_FULL_ATTN_SELECT)), dtype=torch.uint8, device=device)
    O, LSE, idx, _ = hs2.hs2_full_attn_select(prob, q, k, v, ws=ws)
    t_full = med(lambda: hs2.hs2_full_attn_select(prob, q, k, v, out=O, lse=LSE, idx=idx, ws=ws))
    t_att = med(lambda: hs2.hs2_full_attn_select(prob, q, k, v, out=O, lse=LSE, want_idx=False, ws=ws))
    osp = torch.empty_like(q)
    t_sp = med(lambda: hs2.hs2_sparse_attn_prefill(prob, inp.q_sparse[0], k, v, idx, out=osp))
    # the same layer on the e4m3 cache (codes + one fp32 scale per (token, KV head)): 520 B per attended token
    from gen.workloads import quantize_kv_e4m3
    k8, ksc = quantize_kv_e4m3(k)
    v8, vsc = quantize_kv_e4m3(v)
    prob8 = hs2.Problem.from_tensors(q, k8, wl.k_sel, wl.window)
    t_sp8 = med(lambda: hs2.hs2_sparse_attn_prefill_fp8kv(prob8, inp.q_sparse[0], k8, v8, ksc, vsc, idx, out=osp))
    gb = gathered_kv_bytes(wl)
    fl = full_attn_flops(wl)
    out["prefill"] = {
        "workload": "native8k: B=1, L=8192, 64q/1kv heads, D=256, bf16, k=1024, w=128",
        "full_attn_select_ms": round(t_full, 3), "attention_only_ms": round(t_att, 3),
        "attention_tflops": round(fl / (t_att * 1e-3) / 1e12, 1),
        "attention_frac_of_bf16_peak": round(fl / (t_att * 1e-3) / 1e12 / tensor_peak_for(t_att, peaks)[0], 4),
        "attention_peak_kind": tensor_peak_for(t_att, peaks)[1],
        "sparse_prefill_ms": round(t_sp, 3), "gathered_kv_bytes": gb,
        "sparse_prefill_gbs": round(gb / (t_sp * 1e-3) / 1e9, 1),
        "sparse_prefill_frac_of_hbm_peak": round(gb / (t_sp * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
        "fp8_kv_cache": {"sparse_prefill_ms": round(t_sp8, 3), "gathered_kv_bytes": gb / 1024.0 * 520.0,
                         "frac_of_hbm_peak": round(gb / 1024.0 * 520.0 / (t_sp8 * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)},
        "l2": "the 8 MB cache is L2 resident; Q, idx and O (100 MB) stream"}
    del inp, q, k, v, O, LSE, idx, osp, ws, k8, v8, ksc, vsc
    torch.cuda.empty_cache()

    # the same shape at a context of 32K: the full layer (attention + a score sweep of half its flops + top-k) dwarfs the
    # sparse layers, which is the cost structure the hybrid block is built on (Section 3.4)
    from dataclasses import replace
    wl = replace(NATIVE["native8k"], q_len=32768, kv_len=32768, name="native32k")
    inp = make_inputs(wl, device)
    q, k, v = inp.q_full, inp.k, inp.v
    prob = hs2.Problem.from_tensors(q, k, wl.k_sel, wl.window)
    ws = torch.empty(max(256, hs2.hs2_workspace_bytes(prob, binding.HS2_OP_FULL_ATTN_SELECT)), dtype=torch.uint8, device=device)
    O, LSE, idx, _ = hs2.hs2_full_attn_select(prob, q, k, v, ws=ws)
    t_full = med(lambda: hs2.hs2_full_attn_select(prob, q, k, v, out=O, lse=LSE, idx=idx, ws=ws), n=3, warm=1)
    t_att = med(lambda: hs2.hs2_full_attn_select(prob, q, k, v, out=O, lse=LSE, want_idx=False, ws=ws), n=3, warm=1)
    osp = torch.empty_like(q)
    t_sp = med(lambda: hs2.hs2_sparse_attn_prefill(prob, inp.q_sparse[0], k, v, idx, out=osp), n=3, warm=1)
    gb = gathered_kv_bytes(wl)
    fl = full_attn_flops(wl)
    out["prefill_32k"] = {
        "workload": "native32k: B=1, L=32768, 64q/1kv heads, D=256, bf16, k=1024, w=128",
        "full_attn_select_ms": round(t_full, 2), "attention_only_ms": round(t_att, 2),
        "attention_tflops": round(fl / (t_att * 1e-3) / 1e12, 1),
        "attention_frac_of_bf16_peak": round(fl / (t_att * 1e-3) / 1e12 / tensor_peak_for(t_att, peaks)[0], 4),
        "attention_peak_kind": tensor_peak_for(t_att, peaks)[1],
        "sparse_prefill_ms": round(t_sp, 2), "gathered_kv_bytes": gb,
        "sparse_prefill_frac_of_hbm_peak": round(gb / (t_sp * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)}
    del inp, q, k, v, O, LSE, idx, osp, ws
    torch.cuda.empty_cache()

    wl = NATIVE["native_decode"]
    inp = make_inputs(wl, device)
    k, v = inp.k, inp.v
    prob = hs2.Problem.from_tensors(inp.q_full, k, wl.k_sel, wl.window)
    ws_full = torch.empty(max(256, hs2.hs2_workspace_bytes(prob, binding.HS2_OP_FULL_ATTN_SELECT)), dtype=torch.uint8, device=device)
    ws_dec = torch.empty(max(256, hs2.hs2_workspace_bytes(prob, binding.HS2_OP_SPARSE_ATTN_DECODE)), dtype=torch.uint8, device=device)
    nset, burst = 4, 40
    qfs = [inp.q_full] + [torch.randn_like(inp.q_full) for _ in range(nset - 1)]
    idxs, t_full = [], []
    for s in range(nset):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        _, _, idx, _ = hs2.hs2_full_attn_select(prob, qfs[s], k, v, ws=ws_full)
        b.record()
        torch.cuda.synchronize()
        t_full.append(a.elapsed_time(b))
        idxs.append(idx)
    qss = [torch.randn_like(inp.q_full) for _ in range(nset)]
    o1 = torch.empty_like(inp.q_full)

    def run(n):
        for it in range(n):
            hs2.hs2_sparse_attn_decode(prob, qss[it % nset], k, v, idxs[it % nset], out=o1, ws=ws_dec)
    us = med(lambda: run(burst), warm=1) / burst * 1e3
    gb = gathered_kv_bytes(wl)
    k8, ksc = quantize_kv_e4m3(k)
    v8, vsc = quantize_kv_e4m3(v)
    prob8 = hs2.Problem.from_tensors(inp.q_full, k8, wl.k_sel, wl.window)

    def run8(n):
        for it in range(n):
            hs2.hs2_sparse_attn_decode_fp8kv(prob8, qss[it % nset], k8, v8, ksc, vsc, idxs[it % nset], out=o1)
    us8 = med(lambda: run8(burst), warm=1) / burst * 1e3
    ws8 = torch.empty(max(256, hs2.hs2_workspace_bytes(prob8, binding.HS2_OP_FULL_ATTN_SELECT_FP8KV)), dtype=torch.uint8, device=device)
    t_full8 = med(lambda: hs2.hs2_full_attn_select_fp8kv(prob8, qfs[0], k8, v8, ksc, vsc, ws=ws8), n=4, warm=1)
    out["decode_fp8_kv_cache"] = {
        "sparse_decode_us_per_step": round(us8, 2), "gathered_kv_bytes": gb / 1024.0 * 520.0,
        "full_attn_select_decode_ms": round(t_full8, 3),
        "frac_of_hbm_peak": round(gb / 1024.0 * 520.0 / (us8 * 1e-6) / 1e9 / peaks["hbm_gbs"], 4),
        "note": "the FP8 entry point takes no scratch: the splits of a sequence merge inside a thread-block cluster"}
    out["decode"] = {
        "workload": "native_decode: B=64, ctx 65536, 64q/1kv heads, D=256, bf16, k=1024, w=128",
        "sparse_decode_us_per_step": round(us, 2), "gathered_kv_bytes": gb,
        "achieved_gbs": round(gb / (us * 1e-6) / 1e9, 1), "frac_of_hbm_peak": round(gb / (us * 1e-6) / 1e9 / peaks["hbm_gbs"], 4),
        "full_attn_select_decode_ms": round(min(t_full[1:]), 3), "launches_back_to_back": burst,
        "l2": "4.3 GB cache, 4 rotating query/index sets > L2"}
    return out


def bench_kv_project(device, peaks, reps=7):
    """The cache producer (Section 3.2, KV Bridging): C = H W^T for the paper's hidden size 2048 and four layers' K and V
    projections (2048 output columns) over 32768 tokens; bf16 output and the quantising e4m3 output."""
    import paper_2609_26368_b200 as hs2
    T, dm, N = 32768, 2048, 2048
    h = torch.randn(T, dm, device=device).to(torch.bfloat16)
    w = (torch.randn(N, dm, device=device) / dm ** 0.5).to(torch.bfloat16)
    out = torch.empty(T, N, dtype=torch.bfloat16, device=device)
    o8 = torch.empty(T, N, dtype=torch.uint8, device=device)
    sc = torch.empty(T, N // 128, dtype=torch.float32, device=device)

    def med(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)
    fl = 2.0 * T * dm * N
    t16 = med(lambda: hs2.hs2_kv_project(h, w, out=out))
    t8 = med(lambda: hs2.hs2_kv_project(h, w, out=o8, fp8=True, scales=sc))
    peak = peaks.get("bf16_tflops", peaks["bf16_tflops_sustained"])
    tlib = med(lambda: torch.matmul(h, w.t(), out=out))     # the vendor library's GEMM on the same operands, for context only
    return {"workload": "T=32768 tokens, d_model 2048, 2048 output columns, bf16 in, fp32 accumulate",
            "library_gemm_us": round(tlib * 1e3, 1), "library_gemm_tflops": round(fl / tlib / 1e9, 1),
            "bf16_out_us": round(t16 * 1e3, 1), "bf16_out_tflops": round(fl / t16 / 1e9, 1),
            "e4m3_out_us": round(t8 * 1e3, 1), "e4m3_out_tflops": round(fl / t8 / 1e9, 1),
            "peak_tflops_burst": peak, "frac_bf16_out": round(fl / t16 / 1e9 / peak, 4),
            "frac_e4m3_out": round(fl / t8 / 1e9 / peak, 4), "l2": "A, B and C are 134 + 8 + 134 MB: larger than L2"}


# ------------------------------------------------------------------ CPU oracle legs

def oracle_sample_step(wl, inp_host, rows):
    """The oracle, as it stands, on a sample of query rows: full attention + selection + sparse layers."""
    import oracle
    O, LSE, idx, _ = oracle.full_attn_select(inp_host.q_full, inp_host.k, inp_host.v, wl.k_sel, wl.window, rows=rows)
    for q in inp_host.q_sparse:
        oracle.sparse_attn(q, inp_host.k, inp_host.v, idx, wl.window, rows=rows)


def host_inputs(wl):
    """The workload's tensors in host memory (drawn on the GPU when there is one: the generator is counter based, and
    the large configurations take minutes to draw on the host cores)."""
    if torch.cuda.is_available():
        from dataclasses import replace as _r
        inp = make_inputs(wl, "cuda")
        out = _r(inp, q_full=inp.q_full.cpu(), k=inp.k.cpu(), v=inp.v.cpu(), q_sparse=[q.cpu() for q in inp.q_sparse])
        del inp
        torch.cuda.empty_cache()
        return out
    return make_inputs(wl, "cpu")


def rows_for_flops(wl, flops):
    n = int(flops / oracle_row_flops(wl))
    return max(8, min(n, wl.q_len))


def cpu_baseline(wl, n_rows):
    import oracle
    oracle.build()
    inp = host_inputs(wl)
    rows = [(b, i) for b in range(wl.batch) for i in sample_rows(wl, max(1, n_rows // wl.batch))]
    t0 = time.time()
    oracle_sample_step(wl, inp, rows)
    dt = time.time() - t0
    return {"value": round(len(rows) / dt, 3), "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "%d query rows of %s (budget edges + seeded uniform), all heads, full-attn+select+%d sparse "
                      "layer(s), %.1f s" % (len(rows), wl.name, len(inp.q_sparse), dt)}


def run_reference(args, wl):
    """--impl reference: the CPU oracle on a bounded sample of the workload, same metric and unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    inp = host_inputs(wl)
    # a bounded sample per step (about 5e10 flops, two to three seconds on 16 cores), so that K steps end within a
    # few minutes on the machine's host cores
    n = args.cpu_rows if args.cpu_rows > 0 else rows_for_flops(wl, 5e10)
    rows = [(b, i) for b in range(wl.batch) for i in sample_rows(wl, max(1, min(n, 1024) // wl.batch))]
    for _ in range(min(args.warmup, 1)):
        oracle_sample_step(wl, inp, rows[:8])
    t0 = time.time()
    for _ in range(args.steps):
        oracle_sample_step(wl, inp, rows)
    dt = time.time() - t0
    val = args.steps * len(rows) / dt
    sample = "%d sampled query rows of %s per step (all heads)" % (len(rows), wl.name)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(val, 3), "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt / args.steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, 1),
        "cpu_baseline": {"value": round(val, 3), "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": round(val, 3), "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(wl, n_gpus):
    step_mb = (2 + 2 * wl.n_sparse_layers) * wl.batch * wl.q_len * wl.n_q_heads * wl.head_dim * 2 / 1e6 \
        + wl.batch * wl.n_kv_heads * wl.q_len * wl.k_sel * 4 / 1e6
    return {"workload": "%s: B=%d, L=%d, %dq/%dkv heads, D=%d, %s, k=%d, w=%d, 1 full + %d sparse layer(s) + 1 decode step"
                        % (wl.name, wl.batch, wl.q_len, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.dtype,
                           wl.k_sel, wl.window, wl.n_sparse_layers),
            "structure": wl.structure, "sharding": "replica per GPU, no collective in the path (x%d)" % n_gpus,
            "l2": "inputs larger than L2: every step streams %.0f MB of Q, O and idx; the K/V cache of one KV head "
                  "(%.1f MB) is L2 resident while its queries run" % (step_mb, 2 * wl.kv_len * wl.head_dim * 2 / 1e6)}


# ------------------------------------------------------------------ roofline of the sparse-prefill kernel

def sparse_roofline(wl, block, sp_ms, peaks):
    """`frac`: gathered K/V bytes at the HBM peak, as the benchmark defines it (above 1 when the cache is L2
    resident).  `frac_l2`: against the bare gather of the same rows measured now.  `binding_limit`: the slowest of
    (recorded DRAM traffic at the HBM peak, flops at the bf16 peak, the measured gather) over the kernel's time."""
    gb = gathered_kv_bytes(wl)
    ach = gb / (sp_ms * 1e-3) / 1e9
    tokens = wl.batch * wl.q_len
    traffic, traffic_src = NCU_DRAM_TRAFFIC.get(wl.name, (None, None))
    probe_ms, probe_mode = block.gather_ceiling_ms()
    tpeak, which = tensor_peak_for(sp_ms, peaks)
    t_tensor = sparse_attn_flops(wl) / (tpeak * 1e12) * 1e3
    t_dram = traffic / (peaks["hbm_gbs"] * 1e9) * 1e3 if traffic else None
    limits = {"gather_ms": round(probe_ms, 4), "tensor_ms": round(t_tensor, 4),
              "dram_ms": None if t_dram is None else round(t_dram, 4)}
    limit = max(v for v in (probe_ms, t_tensor, t_dram) if v is not None)
    return {"kernel": "k_sparse_prefill (hs2_sparse_attn_prefill)", "bound": "hbm", "achieved": round(ach, 1),
            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(ach / peaks["hbm_gbs"], 4),
            "traffic": traffic, "traffic_source": None if traffic is None else
            "recorded ncu capture (%s), not measured in this run" % traffic_src,
            "peak_source": peaks["source"], "algorithmic_bytes_per_launch": gb, "ms_per_launch": round(sp_ms, 4),
            "tokens_per_s": round(tokens / (sp_ms * 1e-3), 1),
            "l2_gather_ceiling": {"ms": round(probe_ms, 4), "gbs": round(gb / (probe_ms * 1e-3) / 1e9, 1),
                                  "loads": "past L1" if probe_mode == 0 else "through L1",
                                  "ms_past_l1": round(block.probe_ms_by_mode[0], 4),
                                  "ms_through_l1": round(block.probe_ms_by_mode[1], 4),
                                  "frac_of_the_gather_past_l1": round(block.probe_ms_by_mode[0] / sp_ms, 4),
                                  "how": "hs2_probe_gather on the same K, V and idx: every attended row fetched in the "
                                         "attention kernel's item order, no arithmetic, full occupancy"},
            "frac_l2": round(probe_ms / sp_ms, 4),
            "binding_limit": dict(limits, frac=round(limit / sp_ms, 4), tensor_peak=which),
            "note": "achieved counts gathered K/V rows (512 B per attended token per KV head); one KV head's cache is "
                    "L2 resident in prefill, so frac (of the HBM peak) exceeds 1 and is no measure of distance to a "
                    "limit; frac_l2 is (against the faster of the probe's two load modes; the attention kernel itself "
                    "copies past L1, whose capacity its shared memory takes)"}


def full_layer_summary(wl, fa_ms, peaks):
    fl = full_attn_flops(wl)
    tpeak, which = tensor_peak_for(fa_ms, peaks)
    return {"ms": round(fa_ms, 3), "effective_tflops": round(fl / (fa_ms * 1e-3) / 1e12, 2),
            "peak_tflops": tpeak, "peak_kind": which, "frac": round(fl / (fa_ms * 1e-3) / 1e12 / tpeak, 4),
            "note": "causal QK^T+PV flops only; score sweep and top-k are not credited"}


def side_block(name, device, rank, peaks, world, steps=5):
    """A smaller prefill configuration, timed briefly with the same step (side section of the JSON line)."""
    wl = CONFIGS[name]
    block = Block(wl, device, rank)
    ms = time_steps(block, steps, 3, world)
    km = block.kernel_means()
    out = {"workload": workload_config(wl, world)["workload"], "ms_per_step": round(ms / steps, 4),
           "tokens_per_s": round(wl.batch * wl.q_len * steps / (ms * 1e-3), 1),
           "kernel_ms": {k: round(v, 4) for k, v in km.items()}}
    if km.get("sparse_attn_prefill"):
        out["roofline"] = sparse_roofline(wl, block, km["sparse_attn_prefill"], peaks)
    if km.get("full_attn_select"):
        out["full_attn_select"] = full_layer_summary(wl, km["full_attn_select"], peaks)
    del block
    torch.cuda.empty_cache()
    return out


def bench_variants(device, peaks):
    """The sparse layer on an e4m3 cache and the block-level selection of the paper's first ablation (Section 5), both at
    cfg2's shape: measured numbers for the two variants that the block step itself does not run."""
    import paper_2609_26368_b200 as hs2
    from paper_2609_26368_b200 import binding
    from gen.workloads import quantize_kv_e4m3
    wl = CONFIGS["cfg2"]
    inp = make_inputs(wl, device)
    q, k, v = inp.q_full, inp.k, inp.v
    prob = hs2.Problem.from_tensors(q, k, wl.k_sel, wl.window)
    ws = torch.empty(max(256, hs2.hs2_workspace_bytes(prob, binding.HS2_OP_FULL_ATTN_SELECT)), dtype=torch.uint8, device=device)
    _, _, idx, _ = hs2.hs2_full_attn_select(prob, q, k, v, ws=ws)

    def med(fn, n=10, warm=3):
        for _ in range(warm):
            fn()
        ts = []
        for _ in range(n):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)
    out = torch.empty_like(q)
    t_tok = med(lambda: hs2.hs2_full_attn_select(prob, q, k, v, ws=ws))
    t_bf = med(lambda: hs2.hs2_sparse_attn_prefill(prob, inp.q_sparse[0], k, v, idx, out=out))
    k8, ksc = quantize_kv_e4m3(k)
    v8, vsc = quantize_kv_e4m3(v)
    t_f8 = med(lambda: hs2.hs2_sparse_attn_prefill_fp8kv(prob, inp.q_sparse[0], k8, v8, ksc, vsc, idx, out=out))
    pb = hs2.Problem.from_tensors(q, k, wl.k_sel, wl.window, select_block=64)
    wsb = torch.empty(max(256, hs2.hs2_workspace_bytes(pb, binding.HS2_OP_FULL_ATTN_SELECT)), dtype=torch.uint8, device=device)
    _, _, idxb, _ = hs2.hs2_full_attn_select(pb, q, k, v, ws=wsb)
    t_blk = med(lambda: hs2.hs2_full_attn_select(pb, q, k, v, ws=wsb))
    t_sp_blk = med(lambda: hs2.hs2_sparse_attn_prefill(prob, inp.q_sparse[0], k, v, idxb, out=out))
    gb = gathered_kv_bytes(wl)
    # hs2_topk_select on a materialised score tensor [B, Hkv, Lq, Lk] fp32 (the debug scores of the full layer): the
    # kernel reads each row's candidates (keys 0 .. pos - w) once
    del k8, v8, ksc, vsc
    _, _, _, sc = hs2.hs2_full_attn_select(prob, q, k, v, want_scores=True)
    idx2 = torch.empty_like(idx)
    t_topk = med(lambda: hs2.hs2_topk_select(prob, sc, idx=idx2))
    cand_bytes = 4.0 * wl.batch * wl.n_kv_heads * sum(max(0, i - wl.window + 1) for i in range(wl.kv_len - wl.q_len, wl.kv_len))
    same = bool(torch.equal(idx2, idx))
    del sc
    return {"workload": workload_config(wl, 1)["workload"],
            "topk_select": {"ms": round(t_topk, 4), "candidate_bytes": cand_bytes,
                            "achieved_gbs": round(cand_bytes / (t_topk * 1e-3) / 1e9, 1),
                            "frac_of_hbm_peak": round(cand_bytes / (t_topk * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
                            "same_indices_as_full_layer": same,
                            "note": "fp32 scores read once; instruction-bound (about 50 instructions per candidate), not bandwidth-bound"},
            "fp8_kv_cache": {"sparse_prefill_ms": round(t_f8, 4), "bf16_cache_ms": round(t_bf, 4),
                             "gathered_kv_bytes": gb / 512.0 * 264.0,
                             "note": "the cache is L2 resident at this size: the e4m3 rows halve the copies and the shared memory per warp"},
            "block_level_selection": {"block": 64, "full_attn_select_ms": round(t_blk, 4), "token_level_ms": round(t_tok, 4),
                                      "sparse_prefill_on_block_indices_ms": round(t_sp_blk, 4),
                                      "sparse_prefill_on_token_indices_ms": round(t_bf, 4),
                                      "note": "Section 5, Ablation 1: 16 blocks of 64 tokens against 1024 tokens; the sparse kernel is the same, "
                                              "block indices gather contiguous runs of rows"}}


# ------------------------------------------------------------------ main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(CONFIGS))
    ap.add_argument("--cpu-rows", type=int, default=0,
                    help="query rows of the CPU-oracle sample (0: as many as about 3.5e11 oracle flops, 10-20 s)")
    ap.add_argument("--skip", default="", help="comma list of: block, small, decode64k, native, kvproj, variants, e2e, cpu")
    ap.add_argument("--decode-ctx", type=int, default=65536, help="context length of the decode section (profiling: 8192)")
    ap.add_argument("--decode-batch", type=int, default=0, help="profiling captures only: batch of the decode section (default 64)")
    ap.add_argument("--profile-len", type=int, default=0,
                    help="profiling captures only: shorten the workload to this many tokens (same heads, k and w); "
                         "the printed line is then no benchmark result")
    ap.add_argument("--filter-min-keys", type=int, default=0,
                    help="profiling captures only: context length from which the full layer's selection uses the "
                         "filtered path (hs2_set_filter_min_keys); 0 keeps the library's default")
    args = ap.parse_args()
    wl = CONFIGS[args.workload]
    if args.profile_len > 0:
        from dataclasses import replace
        wl = replace(wl, q_len=args.profile_len, kv_len=args.profile_len, name="%s_len%d" % (wl.name, args.profile_len))
    skip = set(s for s in args.skip.split(",") if s)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        respawn_under_torchrun(args.gpus)
    if args.impl == "reference":
        run_reference(args, wl)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hs2 library has no CPU path")
    import paper_2609_26368_b200 as hs2
    hs2.load_library()
    if args.filter_min_keys > 0:
        hs2.hs2_set_filter_min_keys(args.filter_min_keys)
    rank, world, local = dist_setup(args.gpus)
    device = torch.device("cuda", local if world > 1 else 0)
    peaks = measured_peaks()
    warmup = max(args.warmup, 3)

    if "block" in skip:      # side sections only (used for profiling captures)
        side = {}
        if "decode64k" not in skip:
            side["decode_64k"] = bench_decode_64k(device, peaks, ctx=args.decode_ctx, batch=args.decode_batch)
        if "native" not in skip:
            side["paper_native_shape"] = bench_native(device, peaks)
        if "kvproj" not in skip:
            side["kv_project"] = bench_kv_project(device, peaks)
        if "variants" not in skip:
            side["variants_cfg2"] = bench_variants(device, peaks)
        print(json.dumps(side))
        return
    block = Block(wl, device, rank)
    tokens_per_step = wl.batch * wl.q_len

    # ---- device-resident timing
    sampler = ClockSampler(device.index).start() if rank == 0 else None
    t_wall0 = time.time()
    ms = time_steps(block, args.steps, warmup, world)
    t_wall1 = time.time()
    launches_timed = block.launches
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    ms = max_over_ranks(ms, world, device)
    kmeans = block.kernel_means()
    value = world * tokens_per_step * args.steps / (ms * 1e-3)

    # ---- roofline of the sparse-prefill kernel (the metric's kernel), with the gather ceiling measured now
    roofline = None
    if rank == 0 and kmeans.get("sparse_attn_prefill"):
        roofline = sparse_roofline(wl, block, kmeans["sparse_attn_prefill"], peaks)

    # ---- end to end: pinned host inputs in, outputs back, every step
    e2e = None
    if "e2e" not in skip:
        ms_e2e = time_e2e(wl, device, rank, block, args.steps, world)
        ms_e2e = max_over_ranks(ms_e2e, world, device)
        outs = block.output_tensors()
        e2e = {"value": round(world * tokens_per_step * args.steps / (ms_e2e * 1e-3), 1), "unit": "tokens/s",
               "h2d_bytes_per_step": int(block.input_bytes()),
               "d2h_bytes_per_step": int(sum(t.numel() * t.element_size() for t in outs)),
               "ms_per_step": round(ms_e2e / args.steps, 3),
               "pipeline": "two device buffer sets; H2D of step n+1 and D2H of step n-1 overlap the kernels of step n; "
                           "the kernels of a step replay from one CUDA graph per buffer set"}

    if rank != 0:
        return
    kernels = {k: round(v, 4) for k, v in kmeans.items()}
    extra = {}
    if kmeans.get("full_attn_select"):
        extra["full_attn_select"] = full_layer_summary(wl, kmeans["full_attn_select"], peaks)
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": round(ms / args.steps, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic", "config": workload_config(wl, world),
        "clocks": clocks, "gpu_launches": int(launches_timed), "kernel_ms": kernels, "roofline": roofline,
    }
    line.update(extra)
    if e2e:
        line["e2e"] = e2e
    del block
    torch.cuda.empty_cache()
    if "small" not in skip and world == 1:
        for name in ("cfg2", "cfg3"):
            if name != wl.name:
                line[name] = side_block(name, device, rank, peaks, world)
    if "decode64k" not in skip and world == 1:
        line["decode_64k"] = bench_decode_64k(device, peaks, ctx=args.decode_ctx, batch=args.decode_batch)
    if "native" not in skip and world == 1:
        torch.cuda.empty_cache()
        line["paper_native_shape"] = bench_native(device, peaks)
    if "kvproj" not in skip and world == 1:
        torch.cuda.empty_cache()
        line["kv_project"] = bench_kv_project(device, peaks)
    if "variants" not in skip and world == 1:
        torch.cuda.empty_cache()
        line["variants_cfg2"] = bench_variants(device, peaks)
    if "cpu" not in skip and world == 1:
        torch.cuda.empty_cache()
        n = args.cpu_rows if args.cpu_rows > 0 else rows_for_flops(wl, 3.5e11)
        line["cpu_baseline"] = cpu_baseline(wl, n)
    print(json.dumps(line))


if __name__ == "__main__":
    main()
