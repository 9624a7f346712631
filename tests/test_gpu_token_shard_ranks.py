"""Sharding a sequence's TOKENS over ranks, with the product on every step: two gloo ranks (two processes that share
the one GPU; neither launches a kernel that waits for the other) each run libra_decode_attn with libra_set_lse_output
over their own run of every sequence's pages, the (out, lse) pairs are all-gathered through the process group into the
part-major [n_parts][rows][d] layout, libra_merge_parts merges them on the device, and every rank checks the result
against the float64 oracle over the whole sequences."""
import json
import os
import socket
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, os.path.join(sys.argv[1], "tests"))
import numpy as np, torch
import torch.distributed as dist
from oracle import attention_oracle as O
from paper_2606_03077_b200 import binding as lib, workloads as W
import gates
dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{sys.argv[2]}", rank=int(sys.argv[3]), world_size=2)
rank, world = dist.get_rank(), dist.get_world_size()
dev = torch.device("cuda:0")
lens = [700, 33, 1, 0, 5300, 2049]
B, Hq, Hkv, d = len(lens), 8, 2, 128
lens_a, bt, q, k, v = W.random_case(7, B, Hq, Hkv, d, lens)        # same seed on every rank: same inputs
# this rank's part of every sequence: pages [edges[rank], edges[rank + 1]) of its block-table row
bt_r = np.full_like(bt, -1)
lens_r = np.zeros(B, dtype=np.int32)
for b in range(B):
    n_pages = (int(lens_a[b]) + 15) // 16
    edges = [0, (n_pages * 2) // 5, n_pages]
    p0, p1 = edges[rank], edges[rank + 1]
    bt_r[b, :p1 - p0] = bt[b, p0:p1]
    lens_r[b] = max(0, min(int(lens_a[b]), p1 * 16) - p0 * 16)
up = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a)).to(dev)
h = lib.Handle(Hq, Hkv, d, k.shape[0], B, bt.shape[1], plan=lib.PlanParams(0, 1, 4, 256, 256, 64))   # the long part is split
ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
dq, dk, dv, dbt, dl = up(q), up(k), up(v), up(bt_r), up(lens_r)
out = torch.zeros((B * Hq, d), dtype=torch.int16, device=dev)
lse = torch.zeros((B * Hq,), dtype=torch.float32, device=dev)
st = torch.cuda.current_stream().cuda_stream
h.set_lse_output(lse.data_ptr())
h.plan(lens_r, ws.data_ptr(), ws.numel(), st)
h.decode_attn(dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(), out.data_ptr(), st)
torch.cuda.synchronize()
assert h.debug_error_word() == 0
n_split = int(len(h.plan_export()["combine"]))
# the exchange: every rank ends up with all parts, part-major
outs = [torch.zeros((B * Hq, d // 2), dtype=torch.int32) for _ in range(world)]   # bf16 pairs as int32 words on the wire
lses = [torch.zeros((B * Hq,), dtype=torch.float32) for _ in range(world)]
dist.all_gather(outs, out.cpu().view(torch.int32))
dist.all_gather(lses, lse.cpu())
parts_out = torch.stack(outs).view(torch.int16).to(dev)      # [n_parts][rows][d] bf16 bits
parts_lse = torch.stack(lses).to(dev)      # [n_parts][rows]
merged = torch.full((B * Hq, d), 0x7FC0, dtype=torch.int16, device=dev)
merged_lse = torch.full((B * Hq,), float("nan"), dtype=torch.float32, device=dev)
lib.libra_merge_parts(0, parts_out.data_ptr(), parts_lse.data_ptr(), world, B * Hq, d, merged.data_ptr(),
                      merged_lse.data_ptr(), st)
torch.cuda.synchronize()
got = merged.view(torch.bfloat16).float().cpu().numpy().reshape(B, Hq, d)
got_lse = merged_lse.cpu().numpy().reshape(B, Hq)
ref, ref_lse = O.paged_decode_attention(q, k, v, bt, lens_a)
inf = np.isneginf(ref_lse)
res = {"rank": rank, "tokens": int(lens_r.sum()), "split_sequences": n_split,
       "finite": bool(np.all(np.isfinite(got))),
       "stated": gates.stated_violations(got, ref), "tight": gates.tight_violations(got, ref),
       "tight_ratio": gates.tight_ratio(got, ref),
       "lse_inf_ok": bool(np.array_equal(np.isneginf(got_lse), inf)),
       "lse_err": float(np.max(np.abs(got_lse[~inf] - ref_lse[~inf])))}
h.close()
print(json.dumps(res))
dist.destroy_process_group()
"""


def test_two_ranks_decode_their_parts_and_merge_to_the_whole(lib, tmp_path):
    port = _free_port()
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = [subprocess.Popen([sys.executable, str(script), ROOT, str(port), str(r)], stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    done = [p.communicate(timeout=600) for p in procs]
    assert all(p.returncode == 0 for p in procs), [e[-2000:] for _, e in done]
    outs = [json.loads(o.strip().splitlines()[-1]) for o, _ in done]
    assert sum(o["tokens"] for o in outs) == 700 + 33 + 1 + 0 + 5300 + 2049 and all(o["tokens"] > 0 for o in outs)
    assert any(o["split_sequences"] > 0 for o in outs)     # a part went through the split path and its own combine
    for o in outs:
        assert o["finite"] and o["stated"] == 0 and o["tight"] == 0, o
        assert o["lse_inf_ok"] and o["lse_err"] <= 8e-3, o
