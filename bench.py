#!/usr/bin/env python
"""Benchmark of the paged GQA decode-attention path (planner + split-KV decode + combine).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl libra|reference]

One "step" is one pass of the whole path over one batch: libra_plan (host planner) followed by
libra_decode_attn (decode kernel with the combine step inside it).  The headline workload is
`longtail_mix_b256`, the largest of the configurations and a long-tailed one (batch 256, 32 query / 8 KV
heads, head_dim 128, 90 % of the lengths in [512, 4096] and 10 % in [16384, 32768]); the other three
large workloads are measured in the same run and summarised in `roofline.per_workload` (and in full
under "workloads").

metric  = achieved KV bandwidth: algorithmic bytes (K and V of every cached token, bf16, exact
          token count) / time of one step; "steps_per_s" is reported beside it.
value   = inputs resident in HBM.  A region of exactly K back-to-back steps is timed with CUDA events
          (barrier + synchronize on both sides, max over ranks); the region is repeated REGIONS times and
          ms_per_step is the median region / K (best and spread are reported too).
roofline= frac is the decode kernel's own duration (a CUDA event pair around every launch) against the
          measured copy rate; frac_chained is the same bytes over the step spacing of the chained region,
          where consecutive launches overlap (programmatic dependent launch).
e2e     = the same step through libra_decode_attn_host: q, both KV pools, block table and lengths
          start in pinned host memory and the output ends there, copies inside the timed region.
L2      = every workload moves at least 8 x the 126 MB L2 per step, or rotates over several copies of
          its KV pools (see config.l2).

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
MAIN_WORKLOAD = "longtail_mix_b256"
REGIONS = 25   # timed regions of K steps each; the figures are medians over them
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_BYTES_ASSUMED = 126 * 1024 * 1024
# dram__bytes_read.sum + dram__bytes_write.sum of one decode launch divided by its algorithmic bytes, from the ncu
# captures summarised under profiles/ (a constant of those captures, not something this run measures):
# lognormal_b64 374.4 MB / 368.1 MB, straggler_b8 1078.0 MB / 1073.7 MB (full captures); longtail_mix_b256 4834.1 MB /
# 4821.6 MB and shift_b128 5774.0 MB / 5754.9 MB over its cycle of three layouts (one-pass captures of the two byte
# counters at full size).
NCU_TRAFFIC_OVER_ALGORITHMIC = {"lognormal_b64": 374.4e6 / 368.128e6, "straggler_b8": 1078.0e6 / 1073.741824e6,
                                "longtail_mix_b256": 4834.1e6 / 4821.590016e6, "shift_b128": 5774.01e6 / 5754.925056e6}


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
            copies = pool_copies_for(self.w.steps, lay0.kv_bytes)
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

    def step_device_layers(self, stream: int, layers: int) -> None:
        """One device-side plan followed by `layers` decode calls on it: what a model with that many attention layers
        issues per generated token (the lengths, hence the plan, are the same for every layer)."""
        s = self.i % len(self.layouts)
        self.h.plan_device(self.lens_dev[s].data_ptr(), self.w.batch, self.ws.data_ptr(), self.ws.numel(), stream)
        for l in range(layers):
            k, v = self.pools[(self.i + l) % len(self.pools)]
            self.h.decode_attn(self.q.data_ptr(), k.data_ptr(), v.data_ptr(), self.bts[s].data_ptr(),
                               self.lens_dev[s].data_ptr(), self.out.data_ptr(), stream)
        self.i += 1

    def bytes_of_steps(self, i0: int, n: int) -> int:
        """KV bytes of steps i0 .. i0 + n - 1 (a workload with several layouts cycles through them, and their
        sizes differ: the bytes of a region are those of the layouts it actually ran)."""
        L = len(self.layouts)
        full, rem = divmod(n, L)
        b = full * sum(l.kv_bytes for l in self.layouts)
        for j in range(rem):
            b += self.layouts[(i0 + j) % L].kv_bytes
        return int(b)

    def step_decode_only(self, stream: int) -> None:
        """decode + combine on the plan already in the workspace (one layout only)."""
        k, v = self.pools[self.i % len(self.pools)]
        self.i += 1
        self.h.decode_attn(self.q.data_ptr(), k.data_ptr(), v.data_ptr(), self.bts[0].data_ptr(),
                           self.lens_dev[0].data_ptr(), self.out.data_ptr(), stream)

    def timed_regions(self, fn, steps: int, warmup: int, regions: int, barrier=None, world: int = 1, agg_dev=None,
                      stream=None):
        """`regions` timed regions of exactly `steps` back-to-back calls of fn(stream) each, CUDA events on the
        launching stream, barrier + synchronize on both sides of every region; with several ranks a region's time
        is the slowest rank's and its bytes the sum.  Returns (list of (ms, kv bytes), launches of this rank)."""
        torch = self.torch
        ts = stream if stream is not None else torch.cuda.current_stream()
        st = ts.cuda_stream
        with torch.cuda.stream(ts):
            for _ in range(warmup):
                fn(st)
        torch.cuda.synchronize()
        out = []
        n0 = self.h.launch_count()
        for _ in range(regions):
            if barrier:
                barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            i0 = self.i
            torch.cuda.synchronize()
            with torch.cuda.stream(ts):
                e0.record()
                for _ in range(steps):
                    fn(st)
                e1.record()
            torch.cuda.synchronize()
            if barrier:
                barrier()
            ms, b = aggregate_over_ranks(e0.elapsed_time(e1), float(self.bytes_of_steps(i0, steps)), world, agg_dev)
            out.append((ms, b))
        assert self.h.debug_error_word() == 0, "device error word set"
        return out, self.h.launch_count() - n0

    def device_plan_regions(self, steps: int, warmup: int, regions: int, graph: bool, decodes_per_plan: int = 1):
        """The step with the device-side planner (libra_plan_device + decode), issued eagerly or replayed from a CUDA
        graph that holds one step per layout x pool copy; same regime as timed_regions.  Returns ms per step (median)."""
        torch = self.torch
        side = torch.cuda.Stream()
        per_replay = len(self.layouts) * len(self.pools)
        with torch.cuda.stream(side):
            for _ in range(max(warmup, per_replay)):
                self.step_device(side.cuda_stream)
        torch.cuda.synchronize()
        if not graph:
            res, _ = self.timed_regions(self.step_device, steps, 0, regions, stream=side)
            return float(np.median([ms / steps for ms, _ in res])), float(np.median([b / (ms * 1e-3) / 1e9 for ms, b in res]))
        self.i = 0
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for _ in range(per_replay):
                if decodes_per_plan == 1:
                    self.step_device(side.cuda_stream)
                else:
                    self.step_device_layers(side.cuda_stream, decodes_per_plan)
        g.replay()
        torch.cuda.synchronize()
        reps = max(1, steps // (per_replay * decodes_per_plan))
        per, gbs = [], []
        for _ in range(regions):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            with torch.cuda.stream(side):
                e0.record()
                for _ in range(reps):
                    g.replay()
                e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            per.append(ms / (reps * per_replay * decodes_per_plan))
            gbs.append(self.bytes_of_steps(0, reps * per_replay) * decodes_per_plan / (ms * 1e-3) / 1e9)
        assert self.h.debug_error_word() == 0, "device error word set"
        return float(np.median(per)), float(np.median(gbs))

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

    def kernel_times(self, steps: int):
        """The same steps with a CUDA event pair around every kernel (recorded by the library on its stream): the
        decode kernel's own duration, launch by launch, without the overlap of consecutive launches.
        Returns (decode ms per launch, ms after decode per launch, launches, KV bytes of those launches)."""
        torch = self.torch
        st = torch.cuda.current_stream().cuda_stream
        steps = min(steps, 4096)
        i0 = self.i
        self.h.profile_begin()
        for _ in range(steps):
            self.step(st)
        torch.cuda.synchronize()
        d, c, n = self.h.profile_end()
        return d / n, c / n, n, self.bytes_of_steps(i0, n)

    def close(self):
        self.h.close()


def median_gbs(res):
    return float(np.median([b / (ms * 1e-3) / 1e9 for ms, b in res]))


def ceilings_measure(rep: Replica, steps: int, regions: int, step_gbs: float):
    """What the step's read rate is set against, timed in the SAME regime as the step (regions of `steps` chained
    calls, median): the step with the attention math removed (same plan, page walk and tiled copies), and a plain
    streaming read of a contiguous 4 GiB buffer (as many calls per region as take about as long as the step's)."""
    torch = rep.torch
    gat, _ = rep.timed_regions(rep.step_gather_read, steps, 3, regions)
    gat_gbs = median_gbs(gat)
    nbytes = 4 << 30
    buf = torch.zeros(nbytes, dtype=torch.uint8, device=rep.dev)
    region_ms = float(np.median([ms for ms, _ in gat]))
    calls = max(2, int(round(region_ms / (nbytes / 7.2e12 * 1e3))))
    rd = []
    st = torch.cuda.current_stream().cuda_stream
    for r in range(regions + 2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(calls):
            rep.h.debug_stream_read(buf.data_ptr(), nbytes, st)
        e1.record()
        torch.cuda.synchronize()
        if r >= 2:
            rd.append((e0.elapsed_time(e1), float(nbytes) * calls))
    del buf
    rd_gbs = median_gbs(rd)
    return {"regions": regions, "steps_per_region": steps, "read_calls_per_region": calls,
            "page_gather_read_gbs": gat_gbs, "contiguous_read_gbs": rd_gbs,
            "step_frac_of_page_gather_read": step_gbs / gat_gbs, "step_frac_of_contiguous_read": step_gbs / rd_gbs,
            "note": "page_gather_read = libra_debug_gather_read (the decode kernel's plan, grid, block-table walk and "
                    "tiled copies, no math); contiguous_read = libra_debug_stream_read over 4 GiB; both in regions of "
                    "chained calls like the step"}


def measure_workload(rep: Replica, steps: int, warmup: int, regions: int, peak: float, barrier=None, world: int = 1,
                     agg_dev=None, with_ceilings: bool = True, with_device_plan: bool = True):
    """Everything the summary of one workload needs, from one replica: the chained regions, the per-launch kernel
    duration, the read ceilings and the device-planned step."""
    res, launches = rep.timed_regions(rep.step, steps, warmup, regions, barrier, world, agg_dev)
    per_step = np.array([ms / steps for ms, _ in res])
    gbs = np.array([b / (ms * 1e-3) / 1e9 for ms, b in res])
    kv_per_step = float(np.mean([b / steps for _, b in res])) / world
    dec_ms, after_ms, n_prof, prof_bytes = rep.kernel_times(max(steps, 3 * len(rep.layouts)) if steps < 200 else 200)
    kernel_gbs = prof_bytes / n_prof / (dec_ms * 1e-3) / 1e9
    m = {"kv_bytes_per_step": kv_per_step, "ms_per_step": float(np.median(per_step)),
         "ms_per_step_best": float(per_step.min()), "ms_per_step_worst": float(per_step.max()),
         "spread_pct": float((per_step.max() - per_step.min()) / np.median(per_step) * 100.0),
         "regions": regions, "steps_per_region": steps,
         "kv_gbs": float(np.median(gbs)), "kv_gbs_best": float(gbs.max()),
         "frac_chained_of_measured": float(np.median(gbs)) / world / peak,
         "frac_chained_of_8TBs": float(np.median(gbs)) / world / NOMINAL_HBM_GBS,
         "kernel_us_event_pairs": dec_ms * 1e3, "after_decode_us_event_pairs": after_ms * 1e3,
         "kernel_gbs": kernel_gbs, "frac_kernel_of_measured": kernel_gbs / peak,
         "frac_kernel_of_8TBs": kernel_gbs / NOMINAL_HBM_GBS, "kernel_launches_timed": n_prof,
         "launches": int(launches), "pool_copies": len(rep.pools)}
    if world == 1:
        if len(rep.layouts) == 1:   # the plan reused: decode + combine only (a caller whose lengths did not change)
            st = rep.torch.cuda.current_stream().cuda_stream
            rep.h.plan(rep.layouts[0].seq_lens, rep.ws.data_ptr(), rep.ws.numel(), st)
            r2, _ = rep.timed_regions(rep.step_decode_only, steps, 3, regions)
            m["ms_per_step_plan_reused"] = float(np.median([ms / steps for ms, _ in r2]))
        if with_ceilings:
            m["ceilings"] = ceilings_measure(rep, steps, max(5, regions // 2), m["kv_gbs"])
        if with_device_plan:
            e_ms, e_gbs = rep.device_plan_regions(steps, 6, max(5, regions // 2), graph=False)
            g_ms, g_gbs = rep.device_plan_regions(steps, 6, max(5, regions // 2), graph=True)
            l_ms, l_gbs = rep.device_plan_regions(max(steps, 64), 6, max(5, regions // 2), graph=True, decodes_per_plan=32)
            m["device_plan"] = {"ms_per_step_eager": e_ms, "kv_gbs_eager": e_gbs, "ms_per_step_cuda_graph": g_ms,
                                "kv_gbs_cuda_graph": g_gbs, "over_host_plan_us": (g_ms - m["ms_per_step"]) * 1e3,
                                "ms_per_decode_call_32_per_plan": l_ms, "kv_gbs_32_per_plan": l_gbs,
                                "note": "libra_plan_device + decode replayed from a CUDA graph (one step per layout x pool "
                                        "copy); 32_per_plan = one device-side plan serving 32 decode calls, as the 32 "
                                        "attention layers of a model share one step's lengths"}
    return m


def compact(m: dict) -> dict:
    """The per-workload figures that must survive in the top-level line."""
    c = {"kv_gbs": round(m["kv_gbs"], 1), "ms_per_step": round(m["ms_per_step"], 5),
         "frac_of_measured": round(m["frac_chained_of_measured"], 4), "frac_of_8TBs": round(m["frac_chained_of_8TBs"], 4),
         "kernel_us_event_pairs": round(m["kernel_us_event_pairs"], 2),
         "frac_kernel_of_measured": round(m["frac_kernel_of_measured"], 4),
         "frac_kernel_of_8TBs": round(m["frac_kernel_of_8TBs"], 4), "spread_pct": round(m["spread_pct"], 2)}
    if "ceilings" in m:
        c["frac_of_contiguous_read"] = round(m["ceilings"]["step_frac_of_contiguous_read"], 4)
        c["frac_of_page_gather_read"] = round(m["ceilings"]["step_frac_of_page_gather_read"], 4)
    if "device_plan" in m:
        c["device_plan_graph_ms"] = round(m["device_plan"]["ms_per_step_cuda_graph"], 5)
        c["device_plan_32_calls_per_plan_ms"] = round(m["device_plan"]["ms_per_decode_call_32_per_plan"], 5)
    return c


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
    the block shape the library picks by itself against the default large shape forced, on host plans; and the plan
    made on the device, without and with the caller's bound on the lengths (libra_set_length_hint)."""
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
        for label, variant, hint in (("auto_shape", None, None), ("default_shape_forced", (8, 3), None),
                                     ("device_plan", None, 0), ("device_plan_length_hint", None, L)):
            h = rep.binding.Handle(w.num_q_heads, 8, 128, pool, Bn, bts[0].shape[1], device=rep.dev.index or 0)
            if variant:
                h.set_variant(*variant)
            if hint is not None:
                h.set_length_hint(hint)
            ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=rep.dev)

            def step(i):
                if hint is None:
                    h.plan(lens, ws.data_ptr(), ws.numel(), st)
                else:
                    h.plan_device(lens_dev.data_ptr(), Bn, ws.data_ptr(), ws.numel(), st)
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


def few_long_measure(rep: Replica, steps: int = 40, regions: int = 5):
    """The tail end of a rollout: a few long stragglers are all that is still decoding.  Batches of 3 to 26 sequences
    of 12K - 40K tokens, planned with and without the planner's second pass (a plan of fewer than one and a half waves
    of long blocks is made again for twice as many slots), on pools of their own (1.2 M tokens, block tables rotated
    over as many placements as fit)."""
    torch, w = rep.torch, rep.w
    if w.head_dim != 128 or w.num_kv_heads != 8:
        return None
    from numpy.random import Generator, PCG64
    rng = Generator(PCG64(0))
    pool_pages = 75000
    k = torch.randn((pool_pages, 8, 16, 128), device=rep.dev, dtype=torch.bfloat16)
    v = torch.randn((pool_pages, 8, 16, 128), device=rep.dev, dtype=torch.bfloat16)
    st = torch.cuda.current_stream().cuda_stream
    batches = {"12 x 20000": np.full(12, 20000), "20 x 12000": np.full(20, 12000), "6 x 30000": np.full(6, 30000),
               "3 x 40000": np.full(3, 40000), "8 x U[16K,32K]": rng.integers(16384, 32769, 8),
               "26 x U[16K,32K]": rng.integers(16384, 32769, 26), "8 x 32768": np.full(8, 32768),
               "32 x 8192": np.full(32, 8192)}
    res = []
    for name, lens in batches.items():
        lens = lens.astype(np.int32)
        Bn = len(lens)
        npg = (lens.astype(np.int64) + 15) // 16
        need = int(npg.sum())
        copies = max(1, min(8, pool_pages // need))
        ld = int(npg.max())
        perm = rng.permutation(pool_pages)
        bts = []
        for c in range(copies):
            bt = np.full((Bn, ld), -1, np.int32)
            pos = c * need
            for b in range(Bn):
                bt[b, :npg[b]] = perm[pos:pos + npg[b]]
                pos += npg[b]
            bts.append(torch.from_numpy(bt).to(rep.dev))
        dl = torch.from_numpy(lens).to(rep.dev)
        q = torch.randn((Bn, w.num_q_heads, 128), device=rep.dev, dtype=torch.bfloat16)
        out = torch.zeros_like(q)
        row = {"batch": name, "kv_bytes": int(lens.astype(np.int64).sum()) * 8 * 128 * 4}
        for label, refine in (("plain", -1), ("refined", 0)):
            h = rep.binding.Handle(w.num_q_heads, 8, 128, pool_pages, Bn, ld, device=rep.dev.index or 0,
                                   plan=rep.binding.PlanParams(0, 0, 0, 0, 0, 0, refine))
            ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=rep.dev)

            def step(i):
                h.plan(lens, ws.data_ptr(), ws.numel(), st)
                h.decode_attn(q.data_ptr(), k.data_ptr(), v.data_ptr(), bts[i % copies].data_ptr(), dl.data_ptr(),
                              out.data_ptr(), st)
            for i in range(8):
                step(i)
            torch.cuda.synchronize()
            ts = []
            for _ in range(regions):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(steps):
                    step(i)
                e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1) / steps)
            assert h.debug_error_word() == 0, "device error word set"
            ms = float(np.median(ts))
            row[label] = {"ms_per_step": ms, "kv_gbs": row["kv_bytes"] / (ms * 1e-3) / 1e9,
                          "blocks": int(len(h.plan_export()["items"])) * 8}
            h.close()
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
def make_config(name: str, world: int) -> dict:
    """The `config` of the JSON line: what the workload is, the same for both arms."""
    from paper_2606_03077_b200 import workloads as W

    w = W.WORKLOADS[name]
    kv = [W.make_layout(name, s)[0].kv_bytes for s in range(w.steps)]
    copies = pool_copies_for(w.steps, kv[0])
    l2 = (f"every step reads {min(kv) / 1e9:.2f} GB or more of KV, at least {min(kv) / L2_BYTES_ASSUMED:.0f} x the 126 MB L2"
          if copies == 1 else
          f"steps rotate over {copies} copies of the KV pools ({copies * kv[0] / 1e9:.2f} GB live KV vs 126 MB L2)")
    return {"workload": name, "batch": w.batch, "q_heads": w.num_q_heads, "kv_heads": w.num_kv_heads,
            "head_dim": w.head_dim, "page_size": w.page_size, "kv_bytes_per_step": float(np.mean(kv)),
            "parallelism": f"replicas x{world}", "l2": l2,
            "step": "libra_plan + decode kernel (the combine step runs inside it)"}


def pool_copies_for(steps_in_workload: int, kv_bytes: int) -> int:
    """Copies of the KV pools a replica rotates over, so that 4 x L2 of other data passes before a pool is read again."""
    if steps_in_workload > 1 or kv_bytes >= 6 * L2_BYTES_ASSUMED:
        return 1
    return max(1, min(8, -(-4 * L2_BYTES_ASSUMED // max(1, kv_bytes)) + 1))


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
            "config": make_config(args.workload, max(1, args.gpus)),
            "cpu_baseline": {k: t_all[-1][k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "steps_per_s": 1e3 / ms, "gpu_launches": 0,
            "note": "each step times the CPU oracle on a bounded sample of the workload's sequences; ms_per_step "
                    "extrapolates to the whole batch"}
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
    from paper_2606_03077_b200 import workloads as W

    variant = tuple(int(x) for x in args.variant.split(",")) if args.variant else None
    plan = (_b.PlanParams(0, args.ctas_per_sm, args.items_per_slot, 0, 0, 0, args.refine)
            if (args.ctas_per_sm or args.items_per_slot or args.refine) else None)
    peak, peak_src = measured_hbm_peak()
    regions = max(1, args.regions)
    solo = rank == 0 and world == 1

    rep = Replica(args.workload, dev, plan=plan, variant=variant)
    sampler = ClockSampler(local_rank)
    sampler.start()
    m = measure_workload(rep, args.steps, args.warmup, regions, peak, barrier, world, agg_dev,
                         with_ceilings=solo and not args.only_main, with_device_plan=solo and not args.only_main)
    clocks = sampler.stop()

    ratio = NCU_TRAFFIC_OVER_ALGORITHMIC.get(args.workload)
    roofline = {"bound": "hbm", "kernel": "decode_kernel", "achieved": m["kernel_gbs"], "peak": peak, "unit": "GB/s",
                "frac": m["frac_kernel_of_measured"], "frac_kernel": m["frac_kernel_of_measured"],
                "frac_chained": m["frac_chained_of_measured"],
                "frac_kernel_of_8TBs": m["frac_kernel_of_8TBs"], "frac_chained_of_8TBs": m["frac_chained_of_8TBs"],
                "peak_source": peak_src,
                "traffic": (m["kv_bytes_per_step"] * (ratio if ratio else float(np.mean(list(NCU_TRAFFIC_OVER_ALGORITHMIC.values()))))),
                "traffic_source": ("ncu capture of this workload, profiles/" if ratio else
                                   "scaled from the ncu captures of the four large workloads (1.003 - 1.017 x the "
                                   "algorithmic bytes)"),
                "algorithmic_bytes_per_launch": m["kv_bytes_per_step"], "kernel_us": m["kernel_us_event_pairs"],
                "chained_step_us": m["ms_per_step"] * 1e3,
                "timing": "frac / frac_kernel: a CUDA event pair around every decode launch (the kernel's own duration); "
                          "frac_chained: step spacing of the timed region, where consecutive launches overlap",
                "launches_timed": m["kernel_launches_timed"],
                "per_workload": {args.workload: compact(m)}}

    line = {"metric": METRIC, "value": m["kv_gbs"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": make_config(args.workload, world),
            "steps_per_s": 1e3 / m["ms_per_step"] * world,
            "regions": {"count": regions, "steps_each": args.steps, "ms_per_step_median": m["ms_per_step"],
                        "ms_per_step_best": m["ms_per_step_best"], "ms_per_step_worst": m["ms_per_step_worst"],
                        "spread_pct": m["spread_pct"]},
            "frac_of_nominal_8TBs": m["frac_chained_of_8TBs"],
            "frac_of_measured_copy": m["frac_chained_of_measured"],
            "gpu_launches": int(m["launches"]), "clocks": clocks, "roofline": roofline}
    if "ms_per_step_plan_reused" in m:
        line["steps_per_s_plan_reused"] = 1e3 / m["ms_per_step_plan_reused"]
    for key in ("ceilings", "device_plan"):
        if key in m:
            line[key] = m[key]

    if solo:
        k0, v0 = rep.pools[0]
        if not args.no_e2e:
            ms, h2d, d2h, same = e2e_measure(rep, args.e2e_steps)
            line["e2e"] = {"value": rep.layouts[0].kv_bytes / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
                           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
                           "matches_resident_run": same,
                           "note": "libra_decode_attn_host: q, both KV pools, block table, lengths copied from pinned "
                                   "host memory every step, output copied back"}
            line["e2e_resident_kv"] = e2e_resident_kv_measure(rep, 100)
        extras = set(x for x in args.extras.split(",") if x)
        if "early_prefetch" in extras:
            # back-to-back steps with libra_set_early_prefetch: the kernel before each decode launch is the previous
            # step's decode kernel, which writes only `out` and the workspace, so the promise holds
            rep.h.set_early_prefetch(True)
            r_e, _ = rep.timed_regions(rep.step, args.steps, 3, max(5, regions // 2))
            rep.h.set_early_prefetch(False)
            line["early_prefetch"] = {"ms_per_step": float(np.median([ms / args.steps for ms, _ in r_e])),
                                      "kv_gbs": median_gbs(r_e), "note": "optional mode, off in the headline number"}
        n_x = min(200, max(20, args.steps))
        if "multi_token" in extras:
            line["multi_token"] = [x for x in (multi_token_measure(rep, t, n_x) for t in (2, 4)) if x]
        if "fp8_cache" in extras:
            line["fp8_cache"] = fp8_cache_measure(rep, steps=n_x)
        if "nhd_layout" in extras:
            line["nhd_layout"] = nhd_layout_measure(rep, n_x)
        if "head_shard" in extras:
            line["head_shard"] = head_shard_measure(rep, n_x)
        if "wide_group" in extras:
            line["wide_group"] = wide_group_measure(rep, n_x)
        if "short_batch" in extras:
            line["short_batch"] = short_batch_measure(rep)
        if "ring_step" in extras:
            line["ring_step"] = ring_step_measure(rep)
        if "few_long" in extras:
            line["few_long"] = few_long_measure(rep)
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

    if not args.only_main and not args.no_others and world == 1:
        others = {}
        for name in W.WORKLOAD_ORDER[1:]:
            if name == args.workload:
                continue
            r = Replica(name, dev)
            mo = measure_workload(r, args.steps, max(3, args.warmup), regions, peak)
            roofline["per_workload"][name] = compact(mo)
            if args.full:
                n_x = min(60, max(20, args.steps))
                mo["multi_token"] = [x for x in (multi_token_measure(r, t, n_x) for t in (2, 3, 4)) if x]
                mo["fp8_cache"] = fp8_cache_measure(r, n_x)
                mo["nhd_layout"] = nhd_layout_measure(r, n_x)
                mo["head_shard"] = head_shard_measure(r, n_x)
                if name in ("longtail_mix_b256", "straggler_b8"):
                    mo["kv_migration"] = kv_migration_measure(r)
            others[name] = mo
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
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--regions", type=int, default=REGIONS, help="timed regions of --steps steps each (median reported)")
    ap.add_argument("--impl", default="libra", choices=["libra", "reference"])
    ap.add_argument("--workload", default=MAIN_WORKLOAD)
    ap.add_argument("--only-main", action="store_true", help="skip the other workloads, the ceilings and the device plan")
    ap.add_argument("--no-others", action="store_true", help="measure the chosen workload only (with its ceilings and device plan)")
    ap.add_argument("--full", action="store_true", help="the side measurements on every workload, not only the headline")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-budget", type=float, default=20.0, help="seconds of oracle work for cpu_baseline")
    ap.add_argument("--extras", default="early_prefetch,multi_token,fp8_cache,nhd_layout,head_shard,wide_group,short_batch,kv_migration,ring_step,few_long",
                    help="side measurements on the main workload at N=1 (comma list; empty = none)")
    ap.add_argument("--variant", default="", help="warps,stages of the decode block (default: the library's)")
    ap.add_argument("--ctas-per-sm", type=int, default=0, help="planner constant (0 = default)")
    ap.add_argument("--items-per-slot", type=int, default=0, help="planner constant (0 = default)")
    ap.add_argument("--refine", type=int, default=0, help="planner constant (0 = default, -1 = never)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_libra(args)


if __name__ == "__main__":
    main()
