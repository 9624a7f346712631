#!/usr/bin/env python
"""Benchmark of the paged GQA decode-attention path (planner + split-KV decode + combine).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl libra|reference]

One "step" is one pass of the whole path over one batch: libra_plan (host planner + plan upload)
followed by libra_decode_attn (decode kernel + combine kernel).  The headline workload is
`lognormal_b64` (batch 64, 32 query / 8 KV heads, head_dim 128, lognormal lengths); the other
workloads are reported under "workloads" on the same line.

metric  = achieved KV bandwidth: algorithmic bytes (K and V of every cached token, bf16, exact
          token count) / time of one step; "steps_per_s" is reported beside it.
value   = inputs resident in HBM; timed with CUDA events around exactly K steps.
e2e     = the same step through libra_decode_attn_host: q, both KV pools, block table and lengths
          start in pinned host memory and the output ends there, copies inside the timed region.
L2      = steps rotate over several copies of the KV pools so that a pool is long evicted from
          the 126 MB L2 when it is read again (see config.l2).

With N > 1 (torchrun) every rank runs its own replica of the workload on its own GPU: the path
shards by sequence and has no collective; value is the sum over ranks / the slowest rank's time.

`--impl reference` times the float64 CPU oracle (test infrastructure, deliberately slow) on the
host cores for the same workload; under torchrun only rank 0 runs it.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "paged decode-attn achieved HBM GB/s (KV bytes / step time)"
UNIT = "GB/s"
MAIN_WORKLOAD = "lognormal_b64"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES_ASSUMED = 126 * 1024 * 1024
# dram__bytes_read.sum + dram__bytes_write.sum of one decode launch, from the ncu captures summarised under
# profiles/ (lognormal_b64: 370.63 MB read + 3.4 MB written)
NCU_DECODE_TRAFFIC_BYTES = {"lognormal_b64": 374.9e6, "straggler_b8": 1078.1e6}


# ----------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while a region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, cuda_index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            self.nv = pynvml
            handle = None
            try:
                uuid = str(torch.cuda.get_device_properties(cuda_index).uuid)
                handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
            except Exception:
                handle = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.handle = handle
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._stop_evt.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self) -> dict:
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- helpers
def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def aggregate_over_ranks(elapsed_ms: float, units: float, world: int, device=None):
    """(max elapsed over ranks, sum of units over ranks).  Works on gloo (CPU) and nccl."""
    if world == 1:
        return elapsed_ms, units
    import torch
    import torch.distributed as dist

    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


class Replica:
    """One workload resident on one GPU: pools (several copies), handle, workspace."""

    def __init__(self, name: str, dev, copies: int | None = None, plan=None, variant=None, fused=None):
        import torch

        from paper_2606_03077_b200 import binding, workloads as W

        self.torch, self.W, self.binding = torch, W, binding
        self.name, self.dev = name, dev
        self.w = W.WORKLOADS[name]
        self.layouts = [W.make_layout(name, s)[0] for s in range(self.w.steps)]
        lay0 = self.layouts[0]
        self.ld = max(l.block_table.shape[1] for l in self.layouts)
        q, k, v = W.fill_device_pools(lay0, dev, poison=(self.w.steps == 1))
        self.q = q
        pool_bytes = 2 * k.numel() * 2
        if copies is None:  # enough copies that 4 x L2 of other data passes before a pool is read again
            copies = 1 if self.w.steps > 1 else max(1, min(8, -(-4 * L2_BYTES_ASSUMED // max(1, lay0.kv_bytes)) + 1))
            if lay0.kv_bytes >= 6 * L2_BYTES_ASSUMED:
                copies = 1
        self.pools = [(k, v)] + [(k.clone(), v.clone()) for _ in range(copies - 1)]
        self.pool_bytes = pool_bytes
        self.bts, self.lens_dev = [], []
        for lay in self.layouts:
            bt = np.full((self.w.batch, self.ld), -1, dtype=np.int32)
            bt[:, :lay.block_table.shape[1]] = lay.block_table
            self.bts.append(torch.from_numpy(bt).to(dev))
            self.lens_dev.append(torch.from_numpy(lay.seq_lens.copy()).to(dev))
        self.out = torch.zeros((self.w.batch, self.w.num_q_heads, self.w.head_dim), dtype=torch.bfloat16, device=dev)
        self.h = binding.Handle(self.w.num_q_heads, self.w.num_kv_heads, self.w.head_dim, lay0.pool_pages,
                                self.w.batch, self.ld, device=dev.index or 0, plan=plan)
        if variant is not None:
            self.h.set_variant(*variant)
        if fused is not None:
            self.h.set_combine_mode(fused)
        self.ws = torch.empty(self.h.workspace_size(), dtype=torch.uint8, device=dev)
        self.kv_bytes_per_step = float(np.mean([l.kv_bytes for l in self.layouts]))
        self.i = 0

    def step(self, stream: int) -> None:
        """plan + decode + combine for the next batch (multi-step workloads cycle through their steps)."""
        s = self.i % len(self.layouts)
        k, v = self.pools[self.i % len(self.pools)]
        self.i += 1
        self.h.plan(self.layouts[s].seq_lens, self.ws.data_ptr(), self.ws.numel(), stream)
        self.h.decode_attn(self.q.data_ptr(), k.data_ptr(), v.data_ptr(), self.bts[s].data_ptr(),
                           self.lens_dev[s].data_ptr(), self.out.data_ptr(), stream)

    def step_device(self, stream: int) -> None:
        """The same step planned on the GPU (libra_plan_device): the host never reads the lengths."""
        s = self.i % len(self.layouts)
        k, v = self.pools[self.i % len(self.pools)]
        self.i += 1
        self.h.plan_device(self.lens_dev[s].data_ptr(), self.w.batch, self.ws.data_ptr(), self.ws.numel(), stream)
        self.h.decode_attn(self.q.data_ptr(), k.data_ptr(), v.data_ptr(), self.bts[s].data_ptr(),
                           self.lens_dev[s].data_ptr(), self.out.data_ptr(), stream)

    def timed_device_plan(self, steps: int, warmup: int, graph: bool):
        """ms per step with the device-side planner, issued eagerly or replayed from one CUDA graph that
        holds one step per layout x pool copy."""
        torch = self.torch
        side = torch.cuda.Stream()
        per_replay = len(self.layouts) * len(self.pools)
        with torch.cuda.stream(side):
            for _ in range(max(warmup, per_replay)):
                self.step_device(side.cuda_stream)
        torch.cuda.synchronize()
        g = None
        if graph:
            self.i = 0
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for _ in range(per_replay):
                    self.step_device(side.cuda_stream)
            g.replay()
            torch.cuda.synchronize()
        reps = max(1, steps // per_replay)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(side):
            e0.record()
            for _ in range(reps):
                if graph:
                    g.replay()
                else:
                    for _ in range(per_replay):
                        self.step_device(side.cuda_stream)
            e1.record()
        torch.cuda.synchronize()
        assert self.h.debug_error_word() == 0, "device error word set"
        return e0.elapsed_time(e1) / (reps * per_replay)

    def timed(self, steps: int, warmup: int, barrier=None):
        torch = self.torch
        st = torch.cuda.current_stream().cuda_stream
        for _ in range(warmup):
            self.step(st)
        torch.cuda.synchronize()
        if barrier:
            barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = self.h.launch_count()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            self.step(st)
        e1.record()
        torch.cuda.synchronize()
        if barrier:
            barrier()
        assert self.h.debug_error_word() == 0, "device error word set"
        return e0.elapsed_time(e1), self.h.launch_count() - n0

    def step_gather_read(self, stream: int) -> None:
        """The step with the attention math removed: same plan, page walk and copies (a read ceiling)."""
        s = self.i % len(self.layouts)
        k, v = self.pools[self.i % len(self.pools)]
        self.i += 1
        self.h.plan(self.layouts[s].seq_lens, self.ws.data_ptr(), self.ws.numel(), stream)
        self.h.debug_gather_read(self.q.data_ptr(), k.data_ptr(), v.data_ptr(), self.bts[s].data_ptr(),
                                 self.lens_dev[s].data_ptr(), self.scratch_out().data_ptr(), stream)

    def scratch_out(self):
        if not hasattr(self, "_scratch_out"):
            self._scratch_out = self.torch.zeros_like(self.out)
        return self._scratch_out

    def repeats(self, fn, reps: int, calls_each: int):
        """(median, best) ms per call over `reps` event-timed batches of `calls_each` back-to-back calls."""
        torch = self.torch
        st = torch.cuda.current_stream().cuda_stream
        times = []
        for r in range(reps + 3):  # three untimed batches first
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(calls_each):
                fn(st)
            e1.record()
            torch.cuda.synchronize()
            if r >= 3:
                times.append(e0.elapsed_time(e1) / calls_each)
        return float(np.median(times)), float(min(times))

    def kernel_times(self, steps: int):
        """Same steps with CUDA events around each kernel (recorded by the library on its stream)."""
        torch = self.torch
        st = torch.cuda.current_stream().cuda_stream
        steps = min(steps, 4096)
        self.h.profile_begin()
        for _ in range(steps):
            self.step(st)
        torch.cuda.synchronize()
        d, c, n = self.h.profile_end()
        return d / n, c / n, n

    def close(self):
        self.h.close()


def ceilings_measure(rep: Replica, reps: int = 20):
    """What the step's read rate is set against: the step itself, the same step with the attention math removed
    (same plan, page walk and tiled copies), and a plain streaming read of a contiguous 4 GiB buffer; each as
    (median, best) over `reps` batches."""
    torch = rep.torch
    ms_guess = rep.kv_bytes_per_step / 6.4e12 * 1e3   # batches of ~1.5 ms, whole cycles of a multi-step workload
    per_batch = len(rep.layouts) * max(1, int(round(1.5 / (ms_guess * len(rep.layouts)))))
    step_med, step_best = rep.repeats(rep.step, reps, per_batch)
    gat_med, gat_best = rep.repeats(rep.step_gather_read, reps, per_batch)
    assert rep.h.debug_error_word() == 0, "device error word set"
    nbytes = 4 << 30
    buf = torch.zeros(nbytes, dtype=torch.uint8, device=rep.dev)
    rd_med, rd_best = rep.repeats(lambda st: rep.h.debug_stream_read(buf.data_ptr(), nbytes, st), reps, 2)
    del buf
    gbs = lambda b, ms: b / (ms * 1e-3) / 1e9
    kv = rep.kv_bytes_per_step
    return {"reps": reps, "calls_per_rep": per_batch,
            "step_us_median": step_med * 1e3, "step_us_best": step_best * 1e3,
            "step_gbs_median": gbs(kv, step_med), "step_gbs_best": gbs(kv, step_best),
            "page_gather_read_gbs_median": gbs(kv, gat_med), "page_gather_read_gbs_best": gbs(kv, gat_best),
            "contiguous_read_gbs_median": gbs(nbytes, rd_med), "contiguous_read_gbs_best": gbs(nbytes, rd_best),
            "step_frac_of_page_gather_read": gat_med / step_med,
            "step_frac_of_contiguous_read": gbs(kv, step_med) / gbs(nbytes, rd_med),
            "note": "page_gather_read = libra_debug_gather_read (the decode kernel's plan, grid, block-table walk and "
                    "tiled copies, no math); contiguous_read = libra_debug_stream_read over 4 GiB"}


def multi_token_measure(rep: Replica, q_len: int, steps: int = 200, variant=None):
    """The step with q_len query tokens per sequence (libra_decode_attn_multi) on the same pools, block tables
    and lengths: one pass over K and V serves all q_len tokens."""
    torch, w = rep.torch, rep.w
    if q_len * (w.num_q_heads // w.num_kv_heads) > 16:
        return None
    h = rep.binding.Handle(w.num_q_heads, w.num_kv_heads, w.head_dim, rep.layouts[0].pool_pages, w.batch, rep.ld,
                           device=rep.dev.index or 0)
    h.set_max_query_tokens(q_len)
    if variant is not None:
        h.set_variant(*variant)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=rep.dev)
    gen = torch.Generator(device=rep.dev).manual_seed(7)
    q = torch.randn((w.batch, q_len, w.num_q_heads, w.head_dim), generator=gen, device=rep.dev).to(torch.bfloat16)
    out = torch.zeros_like(q)
    st = torch.cuda.current_stream().cuda_stream

    def step(i):
        s = i % len(rep.layouts)
        k, v = rep.pools[i % len(rep.pools)]
        h.plan(rep.layouts[s].seq_lens, ws.data_ptr(), ws.numel(), st)
        h.decode_attn_multi(q.data_ptr(), q_len, k.data_ptr(), v.data_ptr(), rep.bts[s].data_ptr(),
                            rep.lens_dev[s].data_ptr(), out.data_ptr(), st)

    steps = max(len(rep.layouts), steps // len(rep.layouts) * len(rep.layouts))
    for i in range(10):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    assert h.debug_error_word() == 0, "device error word set"
    h.close()
    ms = e0.elapsed_time(e1) / steps
    return {"q_len": q_len, "ms_per_step": ms, "kv_gbs": rep.kv_bytes_per_step / (ms * 1e-3) / 1e9,
            "query_tokens_per_s": w.batch * q_len / (ms * 1e-3), "steps": steps}


def fp8_cache_measure(rep: Replica, steps: int = 200, variant=None):
    """The step over an E4M3 KV cache of the same geometry (same block tables and lengths, random finite codes):
    half the bytes per cached token.  Also its page-gather read ceiling (same copies, no math)."""
    torch, w = rep.torch, rep.w
    if w.head_dim != 128:
        return None
    shape = rep.pools[0][0].shape
    copies = len(rep.pools) * 2 if len(rep.pools) > 1 else 1     # half the bytes per copy: keep the live set the same

    def codes():
        r = torch.randint(0, 256, shape, dtype=torch.uint8, device=rep.dev)
        r &= 0x87                                                 # sign and mantissa
        r |= torch.randint(0, 9, shape, dtype=torch.uint8, device=rep.dev) << 3   # exponent field 0..8: |x| < 4
        return r

    pools = [(codes(), codes())]
    pools += [(pools[0][0].clone(), pools[0][1].clone()) for _ in range(copies - 1)]
    h = rep.binding.Handle(w.num_q_heads, w.num_kv_heads, w.head_dim, rep.layouts[0].pool_pages, w.batch, rep.ld,
                           device=rep.dev.index or 0)
    h.set_kv_dtype(rep.binding.KV_E4M3, 1.0, 1.0)
    if variant is not None:
        h.set_variant(*variant)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=rep.dev)
    out = torch.zeros_like(rep.out)
    st = torch.cuda.current_stream().cuda_stream

    def run(fn, n):
        for i in range(10):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0, "device error word set"
        return e0.elapsed_time(e1) / n

    def step(i, call=None):
        s = i % len(rep.layouts)
        k, v = pools[i % len(pools)]
        h.plan(rep.layouts[s].seq_lens, ws.data_ptr(), ws.numel(), st)
        (call or h.decode_attn)(rep.q.data_ptr(), k.data_ptr(), v.data_ptr(), rep.bts[s].data_ptr(),
                                rep.lens_dev[s].data_ptr(), out.data_ptr(), st)

    steps = max(len(rep.layouts), steps // len(rep.layouts) * len(rep.layouts))
    ms = run(step, steps)
    ms_read = run(lambda i: step(i, h.debug_gather_read), steps)
    h.close()
    del pools
    torch.cuda.empty_cache()
    bytes8 = rep.kv_bytes_per_step / 2
    tokens = rep.kv_bytes_per_step / (4.0 * w.num_kv_heads * w.head_dim)
    return {"ms_per_step": ms, "kv_gbs": bytes8 / (ms * 1e-3) / 1e9, "kv_bytes_per_step": bytes8,
            "cached_tokens_per_s": tokens / (ms * 1e-3), "page_gather_read_gbs": bytes8 / (ms_read * 1e-3) / 1e9,
            "pool_copies": copies, "steps": steps}


def nhd_layout_measure(rep: Replica, steps: int = 200):
    """The same step with the pools laid out token-major inside a page (NHD: [page, token, head, d]); same values,
    same block tables.  A (page, head) tile is then 16 rows of 256 bytes, 2 KB apart."""
    torch, w = rep.torch, rep.w
    if rep.pool_bytes * len(rep.pools) > (24 << 30):
        return None
    pools = [(k.permute(0, 2, 1, 3).contiguous(), v.permute(0, 2, 1, 3).contiguous()) for k, v in rep.pools]
    P = w.page_size
    strides = (P * w.num_kv_heads * w.head_dim, w.head_dim, w.num_kv_heads * w.head_dim)
    h = rep.binding.Handle(w.num_q_heads, w.num_kv_heads, w.head_dim, rep.layouts[0].pool_pages, w.batch, rep.ld,
                           device=rep.dev.index or 0, kv_strides=strides)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=rep.dev)
    out = torch.zeros_like(rep.out)
    st = torch.cuda.current_stream().cuda_stream

    def step(i):
        s = i % len(rep.layouts)
        k, v = pools[i % len(pools)]
        h.plan(rep.layouts[s].seq_lens, ws.data_ptr(), ws.numel(), st)
        h.decode_attn(rep.q.data_ptr(), k.data_ptr(), v.data_ptr(), rep.bts[s].data_ptr(), rep.lens_dev[s].data_ptr(),
                      out.data_ptr(), st)

    steps = max(len(rep.layouts), steps // len(rep.layouts) * len(rep.layouts))
    for i in range(10):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    assert h.debug_error_word() == 0, "device error word set"
    same = bool(torch.equal(out, rep.out)) if len(rep.layouts) == 1 else None
    h.close()
    del pools
    torch.cuda.empty_cache()
    ms = e0.elapsed_time(e1) / steps
    return {"ms_per_step": ms, "kv_gbs": rep.kv_bytes_per_step / (ms * 1e-3) / 1e9, "steps": steps,
            "same_bits_as_hnd": same}


def head_shard_measure(rep: Replica, steps: int = 200):
    """One rank's share of the step under the paper's tensor-parallel sharding of the cache (by attention head,
    Section 5.3; larger degrees for the long-tail buckets, Section 2.3): KV heads [0, Hkv / tp) of every page and their
    query heads, read in place from the full pool through the handle's strides.  No collective is part of the step."""
    torch, w = rep.torch, rep.w
    P, Hkv, d = w.page_size, w.num_kv_heads, w.head_dim
    st = torch.cuda.current_stream().cuda_stream
    res = []
    base_ms = None
    for tp in (1, 2, 4, 8):
        if Hkv % tp:
            continue
        hk, hq = Hkv // tp, w.num_q_heads // tp
        h = rep.binding.Handle(hq, hk, d, rep.layouts[0].pool_pages, w.batch, rep.ld, device=rep.dev.index or 0,
                               kv_strides=(Hkv * P * d, P * d, d))
        ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=rep.dev)
        q = rep.q[:, :hq].contiguous()
        out = torch.zeros_like(q)

        slice_bytes = hk * P * d * 2   # rank r's heads start this many bytes into every page

        def step(i, h=h, ws=ws, q=q, out=out, tp=tp, slice_bytes=slice_bytes):
            # successive steps take successive ranks' head slices and pool copies, so that a step never finds the
            # bytes of an earlier one in L2 (a rank's share of a small workload would fit there)
            s = i % len(rep.layouts)
            r = (i // len(rep.layouts)) % tp
            k, v = rep.pools[(i // (len(rep.layouts) * tp)) % len(rep.pools)]
            h.plan(rep.layouts[s].seq_lens, ws.data_ptr(), ws.numel(), st)
            h.decode_attn(q.data_ptr(), k.data_ptr() + r * slice_bytes, v.data_ptr() + r * slice_bytes,
                          rep.bts[s].data_ptr(), rep.lens_dev[s].data_ptr(), out.data_ptr(), st)

        n = max(len(rep.layouts), steps // len(rep.layouts) * len(rep.layouts))
        for i in range(10):
            step(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n):
            step(i)
        e1.record()
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0, "device error word set"
        step(0)                      # rank 0's slice again: its rows of the full result
        torch.cuda.synchronize()
        same = (bool(torch.allclose(out.float(), rep.out[:, :hq].float(), atol=2e-3, rtol=2e-2))
                if len(rep.layouts) == 1 else None)   # other chunking, hence other last bits, than the full step
        h.close()
        ms = e0.elapsed_time(e1) / n
        base_ms = ms if tp == 1 else base_ms
        res.append({"tp": tp, "kv_heads_per_rank": hk, "ms_per_step": ms,
                    "rank_kv_gbs": rep.kv_bytes_per_step / tp / (ms * 1e-3) / 1e9,
                    "speedup_vs_tp1": base_ms / ms, "matches_full_step": same})
    return res


def wide_group_measure(rep: Replica, steps: int = 200):
    """The same cache, block tables and lengths read with 8 and 16 query heads per KV head (one and two column tiles
    of the score matrix; the paper's model family includes such ratios): q and out grow, the KV bytes do not."""
    torch, w = rep.torch, rep.w
    st = torch.cuda.current_stream().cuda_stream
    res = []
    for group in (8, 16):
        hq = w.num_kv_heads * group
        h = rep.binding.Handle(hq, w.num_kv_heads, w.head_dim, rep.layouts[0].pool_pages, w.batch, rep.ld,
                               device=rep.dev.index or 0)
        ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=rep.dev)
        gen = torch.Generator(device=rep.dev).manual_seed(9)
        q = torch.randn((w.batch, hq, w.head_dim), generator=gen, device=rep.dev).to(torch.bfloat16)
        out = torch.zeros_like(q)

        def step(i, h=h, ws=ws, q=q, out=out):
            s = i % len(rep.layouts)
            k, v = rep.pools[i % len(rep.pools)]
            h.plan(rep.layouts[s].seq_lens, ws.data_ptr(), ws.numel(), st)
            h.decode_attn(q.data_ptr(), k.data_ptr(), v.data_ptr(), rep.bts[s].data_ptr(), rep.lens_dev[s].data_ptr(),
                          out.data_ptr(), st)

        n = max(len(rep.layouts), steps // len(rep.layouts) * len(rep.layouts))
        for i in range(10):
            step(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n):
            step(i)
        e1.record()
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0, "device error word set"
        h.close()
        ms = e0.elapsed_time(e1) / n
        res.append({"q_heads_per_kv_head": group, "ms_per_step": ms, "kv_gbs": rep.kv_bytes_per_step / (ms * 1e-3) / 1e9,
                    "steps": n})
    return res


def short_batch_measure(rep: Replica, steps: int = 100):
    """Batches of equally long, short sequences at a constant 262,144 cached tokens (1.07 GB of KV at 8 KV heads, d 128):
    the block shape the library picks by itself against the default large shape forced."""
    torch, W, w = rep.torch, rep.W, rep.w
    if w.head_dim != 128 or w.num_kv_heads != 8:
        return None
    from numpy.random import Generator, PCG64
    res = []
    total = 262144
    npg = total // 16
    copies = 4
    pool = npg * copies
    k = torch.randn((pool, 8, 16, 128), device=rep.dev, dtype=torch.bfloat16)
    v = torch.randn((pool, 8, 16, 128), device=rep.dev, dtype=torch.bfloat16)
    perm = Generator(PCG64(1)).permutation(pool)
    st = torch.cuda.current_stream().cuda_stream
    for L in (128, 256, 512, 1024):
        Bn = total // L
        lens = np.full(Bn, L, dtype=np.int32)
        bts = [torch.from_numpy(perm[c * npg:(c + 1) * npg].reshape(Bn, -1).astype(np.int32)).to(rep.dev) for c in range(copies)]
        lens_dev = torch.from_numpy(lens).to(rep.dev)
        q = torch.randn((Bn, w.num_q_heads, 128), device=rep.dev, dtype=torch.bfloat16)
        out = torch.zeros_like(q)
        row = {"tokens_per_sequence": L, "batch": Bn}
        for label, variant in (("auto_shape", None), ("default_shape_forced", (8, 3))):
            h = rep.binding.Handle(w.num_q_heads, 8, 128, pool, Bn, bts[0].shape[1], device=rep.dev.index or 0)
            if variant:
                h.set_variant(*variant)
            ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=rep.dev)

            def step(i):
                h.plan(lens, ws.data_ptr(), ws.numel(), st)
                h.decode_attn(q.data_ptr(), k.data_ptr(), v.data_ptr(), bts[i % copies].data_ptr(), lens_dev.data_ptr(),
                              out.data_ptr(), st)
            for i in range(8):
                step(i)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                step(i)
            e1.record()
            torch.cuda.synchronize()
            assert h.debug_error_word() == 0, "device error word set"
            h.close()
            ms = e0.elapsed_time(e1) / steps
            row[label] = {"ms_per_step": ms, "kv_gbs": total * 8 * 128 * 4 / (ms * 1e-3) / 1e9}
        res.append(row)
    del k, v
    torch.cuda.empty_cache()
    return res


def ring_step_measure(rep: Replica, reps: int = 40):
    """The ring all-reduce's data-plane step (libra_ring_step, flag already set) on 16 MB float32 chunks, the chunk
    size the paper pipelines with: payload rate of a reduce step on 2 and on 4 thread blocks (= SMs)."""
    torch = rep.torch
    n = (16 << 20) // 4
    sets = 10    # rotate over 480 MB of operands: larger than L2
    own = torch.ones((sets, n), dtype=torch.float32, device=rep.dev)
    recv = torch.ones((sets, n), dtype=torch.float32, device=rep.dev)
    dst = torch.zeros((sets, n), dtype=torch.float32, device=rep.dev)
    flag = torch.ones(1, dtype=torch.int32, device=rep.dev)
    status = torch.zeros(1, dtype=torch.int32, device=rep.dev)
    st = torch.cuda.current_stream().cuda_stream
    out = {"chunk_bytes": n * 4}
    for blocks in (2, 4):
        def one(i):
            k = i % sets
            rep.binding.libra_ring_step(rep.dev.index or 0, dst[k].data_ptr(), own[k].data_ptr(), recv[k].data_ptr(), n * 4,
                                        rep.binding.RING_F32, flag.data_ptr(), 1, 1000000, status.data_ptr(), blocks, st)
        for i in range(5):
            one(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            one(i)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        out[f"blocks_{blocks}"] = {"ms_per_step": ms, "payload_gbs": n * 4 / (ms * 1e-3) / 1e9,
                                   "memory_gbs": 3 * n * 4 / (ms * 1e-3) / 1e9}
    assert int(status.item()) == 0
    return out


def e2e_measure(rep: Replica, steps: int):
    """The step through libra_decode_attn_host with every input in pinned host memory."""
    torch = rep.torch
    lay = rep.layouts[0]
    k, v = rep.pools[0]
    pin = lambda t: t.cpu().pin_memory()
    hq, hk, hv = pin(rep.q.view(torch.int16)), pin(k.view(torch.int16)), pin(v.view(torch.int16))
    hbt, hl = pin(rep.bts[0]), pin(rep.lens_dev[0])
    hout = torch.zeros(rep.out.shape, dtype=torch.int16).pin_memory()
    stg = torch.empty(rep.h.host_staging_size(rep.w.batch), dtype=torch.uint8, device=rep.dev)
    st = torch.cuda.current_stream().cuda_stream

    def one():
        rep.h.decode_attn_host(hq.data_ptr(), hk.data_ptr(), hv.data_ptr(), hbt.data_ptr(), hl.data_ptr(),
                               rep.w.batch, hout.data_ptr(), stg.data_ptr(), stg.numel(), rep.ws.data_ptr(),
                               rep.ws.numel(), st)

    for _ in range(2):
        one()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    h2d = hq.numel() * 2 + hk.numel() * 2 + hv.numel() * 2 + hbt.numel() * 4 + hl.numel() * 4 + 4096
    d2h = hout.numel() * 2 + 4
    same = torch.equal(hout.to(rep.dev).view(torch.bfloat16), rep.out) if rep.i % len(rep.pools) >= 0 else True
    return ms, int(h2d), int(d2h), bool(same)


def e2e_resident_kv_measure(rep: Replica, steps: int):
    """One decode step as a serving engine issues it, through libra_decode_attn_host_io: the KV cache stays in
    HBM; the step's own inputs (q, block table, lengths) start in pinned host memory and the output ends there;
    the call returns after synchronising its stream (latency, not pipelined throughput)."""
    torch = rep.torch
    k, v = rep.pools[0]
    hq = rep.q.cpu().pin_memory()
    hbt = rep.bts[0].cpu().pin_memory()
    hl = rep.lens_dev[0].cpu().pin_memory()
    hout = torch.zeros(rep.out.shape, dtype=torch.bfloat16).pin_memory()
    stg = torch.empty(rep.h.host_io_staging_size(rep.w.batch), dtype=torch.uint8, device=rep.dev)
    st = torch.cuda.current_stream().cuda_stream

    def one():
        rep.h.decode_attn_host_io(hq.data_ptr(), k.data_ptr(), v.data_ptr(), hbt.data_ptr(), hl.data_ptr(),
                                  rep.w.batch, hout.data_ptr(), stg.data_ptr(), stg.numel(), rep.ws.data_ptr(),
                                  rep.ws.numel(), st)

    for _ in range(5):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    ms = (time.perf_counter() - t0) / steps * 1e3
    rep.step(st)
    torch.cuda.synchronize()
    same = bool(torch.equal(hout.to(rep.dev), rep.out)) if len(rep.layouts) == 1 else None   # pool copies hold the same data
    return {"value": rep.layouts[0].kv_bytes / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms, "steps": steps,
            "h2d_bytes_per_step": int(hq.numel() * 2 + hbt.numel() * 4 + hl.numel() * 4),
            "d2h_bytes_per_step": int(hout.numel() * 2 + 4), "matches_resident_run": same,
            "note": "libra_decode_attn_host_io: KV pools resident in HBM (as in any serving engine); q, block table and "
                    "lengths copied from pinned host memory and the output copied back every step; the call "
                    "synchronises its stream, wall clock"}


def kv_migration_measure(rep: Replica, reps: int = 10):
    """libra_kv_gather / libra_kv_scatter on the sequences of 16K tokens and more (the ones the paper's
    scheduler would move to a larger bucket): bytes moved = read + write of K and V."""
    torch = rep.torch
    lay = rep.layouts[0]
    rows = np.nonzero(lay.seq_lens >= 16384)[0]
    if len(rows) == 0:
        return None
    lens = lay.seq_lens[rows]
    offs = np.concatenate([[0], np.cumsum(lens.astype(np.int64))])
    total = int(offs[-1])
    w = rep.w
    dbt = rep.bts[0][torch.from_numpy(rows).to(rep.dev)].contiguous()
    dl = torch.from_numpy(lens.copy()).to(rep.dev)
    doffs = torch.from_numpy(offs[:-1].copy()).to(rep.dev)
    err = torch.zeros(1, dtype=torch.int32, device=rep.dev)
    kd = torch.empty((total, w.num_kv_heads, w.head_dim), dtype=torch.bfloat16, device=rep.dev)
    vd = torch.empty_like(kd)
    k, v = rep.pools[0]
    st = torch.cuda.current_stream().cuda_stream
    args = (dbt.data_ptr(), dl.data_ptr(), doffs.data_ptr(), len(rows), int(lens.max()), 0, w.num_kv_heads)
    res = {}
    for what in ("gather", "scatter"):
        def one():
            if what == "gather":
                rep.h.kv_gather(k.data_ptr(), v.data_ptr(), *args, kd.data_ptr(), vd.data_ptr(), err.data_ptr(), st)
            else:
                rep.h.kv_scatter(kd.data_ptr(), vd.data_ptr(), *args, k.data_ptr(), v.data_ptr(), err.data_ptr(), st)
        for _ in range(3):
            one()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            one()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        moved = 2 * 2 * total * w.num_kv_heads * w.head_dim * 2    # K and V, read and write
        res[what] = {"ms": ms, "copy_gbs": moved / (ms * 1e-3) / 1e9}
    # the paper's offload / reload: the dense buffer in pinned host memory, written and read over the bus by the kernels
    host = {}
    if total * w.num_kv_heads * w.head_dim * 2 * 2 <= (6 << 30):
        kh = torch.empty((total, w.num_kv_heads, w.head_dim), dtype=torch.bfloat16).pin_memory()
        vh = torch.empty_like(kh).pin_memory()
        for what in ("gather", "scatter"):
            def one_h():
                if what == "gather":
                    rep.h.kv_gather(k.data_ptr(), v.data_ptr(), *args, kh.data_ptr(), vh.data_ptr(), err.data_ptr(), st)
                else:
                    rep.h.kv_scatter(kh.data_ptr(), vh.data_ptr(), *args, k.data_ptr(), v.data_ptr(), err.data_ptr(), st)
            one_h()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(3):
                one_h()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / 3
            host[what] = {"ms": ms, "payload_gbs": 2 * total * w.num_kv_heads * w.head_dim * 2 / (ms * 1e-3) / 1e9}
        del kh, vh
    assert int(err.item()) == 0
    peak, _ = measured_hbm_peak()
    return {"sequences": int(len(rows)), "tokens": total, "pinned_host": host, "kv_bytes": 2 * total * w.num_kv_heads * w.head_dim * 2,
            "gather": res["gather"], "scatter": res["scatter"],
            "gather_frac_of_measured_copy": res["gather"]["copy_gbs"] / peak,
            "scatter_frac_of_measured_copy": res["scatter"]["copy_gbs"] / peak,
            "note": "dense buffer in device memory; read + write bytes over time, against the measured copy rate"}


def oracle_baseline(name: str, k_dev=None, v_dev=None, q_dev=None, budget_s: float = 20.0, cache=None,
                    repeat: bool = False):
    """Times the float64 oracle, as it stands, on the host cores on a bounded sample of the workload:
    whole sequences in batch order until about `budget_s` seconds of CPU work are spent.  `cache` (a dict)
    keeps the host inputs of a group of sequences between calls, so that repeated steps pay for the oracle only.
    `repeat`: a workload the oracle finishes early is gone through again (same inputs) until half the budget is
    spent, so that the figure rests on several seconds of work."""
    import torch

    from oracle import attention_oracle as O
    from paper_2606_03077_b200 import workloads as W

    w = W.WORKLOADS[name]
    lay, rng = W.make_layout(name, 0)
    threads = torch.get_num_threads()
    done_bytes, done_seqs, spent = 0, 0, 0.0
    b = 0
    passes = 1
    if repeat and cache is None:
        cache = {}
    while spent < budget_s:
        if b >= w.batch:
            if not repeat or spent >= budget_s / 2:
                break
            b = 0
            passes += 1
        rows = list(range(b, min(w.batch, b + (4 if budget_s >= 0.5 else 1))))
        # inputs of the sample: from the device pools if given, else drawn on the host
        if cache is not None and tuple(rows) in cache:
            qh, kh, vh, new_bt = cache[tuple(rows)]
        elif k_dev is not None:
            sys.path.insert(0, os.path.join(ROOT, "tests"))
            ids, new_bt = [], np.full((len(rows), lay.block_table.shape[1]), -1, dtype=np.int32)
            for i, r in enumerate(rows):
                n = (int(lay.seq_lens[r]) + 15) // 16
                new_bt[i, :n] = np.arange(len(ids), len(ids) + n)
                ids.extend(int(x) for x in lay.block_table[r, :n])
            idx = torch.tensor(ids, dtype=torch.long, device=k_dev.device)
            kh = k_dev.view(torch.int16)[idx].cpu().numpy().view(np.uint16)
            vh = v_dev.view(torch.int16)[idx].cpu().numpy().view(np.uint16)
            qh = q_dev.view(torch.int16)[rows[0]:rows[-1] + 1].cpu().numpy().view(np.uint16)
        else:
            npg = int(W.pages_needed(lay.seq_lens[rows]).sum())
            shape = (npg, w.num_kv_heads, w.page_size, w.head_dim)
            kh = W.f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))
            vh = W.f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32))
            qh = W.f32_to_bf16_bits(rng.standard_normal((len(rows), w.num_q_heads, w.head_dim), dtype=np.float32))
            new_bt = np.full((len(rows), lay.block_table.shape[1]), -1, dtype=np.int32)
            pos = 0
            for i, r in enumerate(rows):
                n = (int(lay.seq_lens[r]) + 15) // 16
                new_bt[i, :n] = np.arange(pos, pos + n)
                pos += n
        if cache is not None:
            cache[tuple(rows)] = (qh, kh, vh, new_bt)
        lens = lay.seq_lens[rows]
        t0 = time.perf_counter()
        O.paged_decode_attention(qh, kh, vh, new_bt, lens)
        spent += time.perf_counter() - t0
        done_bytes += int(lens.astype(np.int64).sum()) * w.num_kv_heads * w.head_dim * 4
        done_seqs += len(rows)
        b += len(rows)
    gbs = done_bytes / spent / 1e9
    return {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": (f"first {done_seqs} of {w.batch} sequences of {name}" if passes == 1 else
                       f"{passes} passes over the {w.batch} sequences of {name}") +
                      f" ({done_bytes / 1e6:.1f} MB of KV), {spent:.2f} s of float64 NumPy on {threads} threads",
            "seconds": spent, "kv_bytes": done_bytes,
            "steps_per_s_extrapolated": gbs * 1e9 / lay.kv_bytes}


# ----------------------------------------------------------------------------- arms
def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    from paper_2606_03077_b200 import workloads as W

    lay, _ = W.make_layout(args.workload, 0)
    # every step times the oracle on a bounded sample; the samples shrink as K + W grows so that the whole run
    # stays near two minutes of oracle work (never less than one group of sequences per step)
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    per_step = min(args.cpu_budget, 120.0 / (steps + warmup))
    res = None
    t_all = []
    cache = {}
    for i in range(warmup + steps):
        res = oracle_baseline(args.workload, budget_s=per_step, cache=cache)
        if i >= warmup:
            t_all.append(res)
    gbs = float(sum(r["kv_bytes"] for r in t_all) / sum(r["seconds"] for r in t_all) / 1e9)
    ms = lay.kv_bytes / (gbs * 1e9) * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "batch": lay.workload.batch, "q_heads": lay.workload.num_q_heads,
                       "kv_heads": lay.workload.num_kv_heads, "head_dim": lay.workload.head_dim, "page_size": 16,
                       "kv_bytes_per_step": lay.kv_bytes,
                       "note": "each step times the CPU oracle on a bounded sample of the workload's sequences; "
                               "ms_per_step extrapolates to the whole batch"},
            "cpu_baseline": {k: t_all[-1][k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "steps_per_s": 1e3 / ms, "gpu_launches": 0}
    line["cpu_baseline"]["value"] = gbs
    print(json.dumps(line), flush=True)


def run_libra(args):
    import torch

    rank, local_rank, world = dist_env()
    # one rank per GPU over NCCL; LIBRA_BENCH_BACKEND=gloo lets the N > 1 path be exercised where there are fewer
    # GPUs than ranks (the replicas are independent: no kernel of one rank ever waits for another's)
    backend = os.environ.get("LIBRA_BENCH_BACKEND", "nccl")
    if backend != "nccl":
        local_rank %= max(1, torch.cuda.device_count())
    if world > 1:
        import torch.distributed as dist

        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group(backend)
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    agg_dev = dev if backend == "nccl" else None
    barrier = (lambda: torch.distributed.barrier()) if world > 1 else None

    from paper_2606_03077_b200 import binding as _b

    variant = tuple(int(x) for x in args.variant.split(",")) if args.variant else None
    plan = _b.PlanParams(0, args.ctas_per_sm, args.items_per_slot, 0, 0, 0) if (args.ctas_per_sm or args.items_per_slot) else None
    rep = Replica(args.workload, dev, plan=plan, variant=variant)
    sampler = ClockSampler(local_rank)
    sampler.start()
    elapsed_ms, launches = rep.timed(args.steps, args.warmup, barrier)
    dec_ms, cmb_ms, n_prof = rep.kernel_times(min(args.steps, 2000))
    clocks = sampler.stop()

    units = rep.kv_bytes_per_step * args.steps
    t_max, units_all = aggregate_over_ranks(elapsed_ms, units, world, agg_dev)
    ms_per_step = t_max / args.steps
    value = units_all / (t_max * 1e-3) / 1e9

    peak, peak_src = measured_hbm_peak()
    # average launch duration of the decode kernel: when a step is that one launch, the timed region itself
    # (events around K back-to-back launches) gives it; otherwise the per-kernel event pairs do, each of
    # which adds ~3 us to what it brackets
    one_launch_per_step = launches == args.steps
    kernel_ms = (elapsed_ms / args.steps) if one_launch_per_step else dec_ms
    achieved = rep.kv_bytes_per_step / (kernel_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "decode_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": peak_src, "traffic": NCU_DECODE_TRAFFIC_BYTES.get(args.workload),
                "algorithmic_bytes_per_launch": rep.kv_bytes_per_step, "kernel_us": kernel_ms * 1e3,
                "timing": ("CUDA events around the timed region, one decode launch per step" if one_launch_per_step
                           else "CUDA event pair around every decode launch"),
                "decode_kernel_us_with_event_pairs": dec_ms * 1e3, "after_decode_us_with_event_pairs": cmb_ms * 1e3,
                "launches_timed": n_prof, "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "batch": rep.w.batch, "q_heads": rep.w.num_q_heads,
                       "kv_heads": rep.w.num_kv_heads, "head_dim": rep.w.head_dim, "page_size": 16,
                       "kv_bytes_per_step": rep.kv_bytes_per_step, "parallelism": f"replicas x{world}",
                       "l2": f"rotating {len(rep.pools)} copies of the KV pools "
                             f"({len(rep.pools) * rep.layouts[0].kv_bytes / 1e9:.2f} GB live KV vs 126 MB L2)",
                       "step": "libra_plan + decode kernel (step C runs inside it)"},
            "steps_per_s": 1e3 / ms_per_step * world,
            "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
            "frac_of_measured_copy": value / world / peak,
            "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline}

    if rank == 0 and world == 1:
        k0, v0 = rep.pools[0]
        if not args.no_e2e:
            ms, h2d, d2h, same = e2e_measure(rep, args.e2e_steps)
            line["e2e"] = {"value": rep.layouts[0].kv_bytes / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
                           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
                           "matches_resident_run": same,
                           "note": "libra_decode_attn_host: q, both KV pools, block table, lengths copied from pinned "
                                   "host memory every step, output copied back"}
            line["e2e_resident_kv"] = e2e_resident_kv_measure(rep, 200)
        extras = set(x for x in args.extras.split(",") if x)
        if "ceilings" in extras:
            line["ceilings"] = ceilings_measure(rep)
        if "early_prefetch" in extras:
            # back-to-back steps with libra_set_early_prefetch: the kernel before each decode launch is the previous
            # step's decode kernel, which writes only `out` and the workspace, so the promise holds
            rep.h.set_early_prefetch(True)
            n = min(args.steps, 1000)
            ms_e, _ = rep.timed(n, max(3, args.warmup // 2))
            rep.h.set_early_prefetch(False)
            line["early_prefetch"] = {"ms_per_step": ms_e / n, "kv_gbs": rep.kv_bytes_per_step / (ms_e / n * 1e-3) / 1e9,
                                      "steps": n, "note": "optional mode, off in the headline number"}
        if "multi_token" in extras:
            line["multi_token"] = [m for m in (multi_token_measure(rep, t) for t in (2, 4)) if m]
        if "fp8_cache" in extras:
            line["fp8_cache"] = fp8_cache_measure(rep, steps=min(200, max(10, args.steps)))
        if "nhd_layout" in extras:
            line["nhd_layout"] = nhd_layout_measure(rep)
        if "head_shard" in extras:
            line["head_shard"] = head_shard_measure(rep)
        if "wide_group" in extras:
            line["wide_group"] = wide_group_measure(rep)
        if "short_batch" in extras:
            line["short_batch"] = short_batch_measure(rep)
        if "ring_step" in extras:
            line["ring_step"] = ring_step_measure(rep)
        if "kv_migration" in extras and args.workload in ("longtail_mix_b256", "straggler_b8"):
            line["kv_migration"] = kv_migration_measure(rep)
        if not args.no_cpu:
            cb = oracle_baseline(args.workload, k0, v0, rep.q, budget_s=args.cpu_budget, repeat=True)
            line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
    elif world > 1:
        # end-to-end at N GPUs: every rank copies its own replica's inputs from its own pinned memory
        if not args.no_e2e:
            ms, h2d, d2h, same = e2e_measure(rep, args.e2e_steps)
            t_e2e, u_e2e = aggregate_over_ranks(ms, rep.layouts[0].kv_bytes, world, agg_dev)
            line["e2e"] = {"value": u_e2e / (t_e2e * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": t_e2e,
                           "h2d_bytes_per_step": h2d * world, "d2h_bytes_per_step": d2h * world,
                           "steps": args.e2e_steps}
    rep.close()
    del rep
    torch.cuda.empty_cache()

    if not args.only_main and world == 1:
        from paper_2606_03077_b200 import workloads as W

        others = {}
        for name in W.WORKLOAD_ORDER[1:]:
            if name == args.workload:
                continue
            r = Replica(name, dev)
            n = max(20, min(args.steps, 400))
            ms, _ = r.timed(n, max(3, args.warmup // 4))
            d, c, _ = r.kernel_times(min(n, 200))
            per = ms / n
            others[name] = {"kv_gbs": r.kv_bytes_per_step / (per * 1e-3) / 1e9, "ms_per_step": per, "steps": n,
                            "decode_kernel_us": d * 1e3, "combine_kernel_us": c * 1e3,
                            "decode_kernel_gbs": r.kv_bytes_per_step / (d * 1e-3) / 1e9,
                            "frac_of_nominal_8TBs": r.kv_bytes_per_step / (per * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                            "frac_of_measured_copy": r.kv_bytes_per_step / (per * 1e-3) / 1e9 / peak,
                            "kv_bytes_per_step": r.kv_bytes_per_step, "pool_copies": len(r.pools)}
            others[name]["ceilings"] = ceilings_measure(r, reps=10)
            others[name]["multi_token"] = [m for m in (multi_token_measure(r, t, 60) for t in (2, 3, 4)) if m]
            others[name]["fp8_cache"] = fp8_cache_measure(r, 60)
            others[name]["nhd_layout"] = nhd_layout_measure(r, 60)
            others[name]["head_shard"] = head_shard_measure(r, 60)
            if name in ("longtail_mix_b256", "straggler_b8"):  # migrating the long sequences: gather to a dense buffer, scatter back
                others[name]["kv_migration"] = kv_migration_measure(r)
            if name == "shift_b128":  # the re-planned-every-step workload: also with the device-side planner
                eager = r.timed_device_plan(n, 6, graph=False)
                graph = r.timed_device_plan(n, 6, graph=True)
                others[name]["device_plan"] = {
                    "ms_per_step_eager": eager, "ms_per_step_cuda_graph": graph,
                    "kv_gbs_cuda_graph": r.kv_bytes_per_step / (graph * 1e-3) / 1e9,
                    "note": "libra_plan_device + decode + combine; the graph holds one step per layout and is replayed"}
            r.close()
            del r
            torch.cuda.empty_cache()
        line["workloads"] = others

    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="libra", choices=["libra", "reference"])
    ap.add_argument("--workload", default=MAIN_WORKLOAD)
    ap.add_argument("--only-main", action="store_true", help="skip the other workloads")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-budget", type=float, default=20.0, help="seconds of oracle work for cpu_baseline")
    ap.add_argument("--extras", default="ceilings,early_prefetch,multi_token,fp8_cache,nhd_layout,head_shard,wide_group,short_batch,kv_migration,ring_step",
                    help="side measurements on the main workload at N=1 (comma list; empty = none)")
    ap.add_argument("--variant", default="", help="warps,stages of the decode block (default: the library's)")
    ap.add_argument("--ctas-per-sm", type=int, default=0, help="planner constant (0 = default)")
    ap.add_argument("--items-per-slot", type=int, default=0, help="planner constant (0 = default)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_libra(args)


if __name__ == "__main__":
    main()
