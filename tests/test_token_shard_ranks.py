"""The exchange step of sharding a sequence's TOKENS over ranks, on CPU with two gloo ranks.  What this file checks is
the ORACLE's merge identity and the layout of the exchange only: each rank evaluates the attention over its own run of
pages with the oracle, the (out, lse) pairs are all-gathered into the part-major [n_parts][rows][d] layout that
libra_merge_parts takes, and the oracle's log-sum-exp merge of the gathered pairs is the attention over the whole
sequence.  The library's own step (decode with libra_set_lse_output per rank, libra_merge_parts on the gathered
pairs) runs with two ranks in tests/test_gpu_token_shard_ranks.py and on one process in tests/test_gpu_lse.py."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import numpy as np, torch
import torch.distributed as dist
from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W
dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{sys.argv[2]}", rank=int(sys.argv[3]), world_size=2)
rank, world = dist.get_rank(), dist.get_world_size()
lens = [700, 33, 1, 0, 1300]
B, Hq, Hkv, d = len(lens), 8, 2, 64
lens_a, bt, q, k, v = W.random_case(7, B, Hq, Hkv, d, lens)        # same seed on every rank: same inputs
# this rank's part of every sequence: pages [cut[r], cut[r + 1]) of its block-table row
bt_r = np.full_like(bt, -1)
lens_r = np.zeros(B, dtype=np.int32)
for b in range(B):
    n_pages = (int(lens_a[b]) + 15) // 16
    edges = [0, (n_pages * 2) // 5, n_pages]
    p0, p1 = edges[rank], edges[rank + 1]
    bt_r[b, :p1 - p0] = bt[b, p0:p1]
    lens_r[b] = max(0, min(int(lens_a[b]), p1 * 16) - p0 * 16)
out_r, lse_r = O.paged_decode_attention(q, k, v, bt_r, lens_r)
outs = [torch.zeros(B * Hq, d, dtype=torch.float64) for _ in range(world)]
lses = [torch.zeros(B * Hq, dtype=torch.float64) for _ in range(world)]
dist.all_gather(outs, torch.from_numpy(out_r.reshape(B * Hq, d).copy()))
dist.all_gather(lses, torch.from_numpy(lse_r.reshape(B * Hq).copy()))
parts_out = torch.stack(outs).numpy()      # [n_parts][rows][d]
parts_lse = torch.stack(lses).numpy()      # [n_parts][rows]
ref, ref_lse = O.paged_decode_attention(q, k, v, bt, lens_a)
ref, ref_lse = ref.reshape(B * Hq, d), ref_lse.reshape(B * Hq)
worst, worst_lse = 0.0, 0.0
for r in range(B * Hq):
    o, l = O.merge_partials(parts_out[:, r], parts_lse[:, r])
    worst = max(worst, float(np.max(np.abs(o - ref[r]))))
    if np.isneginf(ref_lse[r]):
        assert np.isneginf(l)
    else:
        worst_lse = max(worst_lse, abs(l - ref_lse[r]))
print(json.dumps({"rank": rank, "tokens": int(lens_r.sum()), "worst": worst, "worst_lse": worst_lse}))
dist.destroy_process_group()
"""


def test_two_ranks_gather_and_merge_to_the_whole(tmp_path):
    port = _free_port()
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = [subprocess.Popen([sys.executable, str(script), ROOT, str(port), str(r)], stdout=subprocess.PIPE, text=True)
             for r in range(2)]
    outs = [json.loads(p.communicate(timeout=300)[0].strip().splitlines()[-1]) for p in procs]
    assert all(p.returncode == 0 for p in procs)
    assert sum(o["tokens"] for o in outs) == 700 + 33 + 1 + 0 + 1300 and all(o["tokens"] > 0 for o in outs)
    for o in outs:
        assert o["worst"] <= 1e-12 and o["worst_lse"] <= 1e-12
