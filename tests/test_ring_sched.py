"""The host side of the ring all-reduce (membership descriptor + schedule, csrc/ring_sched.cpp) on CPU.

* membership edits: a dead peer is taken out, a joining one is put in, neighbours follow;
* the schedules of all members fit together (what one sends in a step is what its successor receives, piece by piece)
  and, executed with NumPy, give the oracle's result bit for bit - so the order of additions is the ring's;
* three gloo ranks (processes): one all-reduce with everybody, then one rank stops joining; the others notice on the host
  (its ready key never appears before the heartbeat timeout), edit the descriptor and all-reduce between themselves.
  No GPU anywhere: the data plane here is NumPy over gloo send / recv, driven by the library's schedule records."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

from oracle import ring_oracle as R

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_membership_edits(lib):
    ring = lib.libra_ring_init([10, 20, 30, 40])
    assert ring.n_members == 4 and list(ring.members[:4]) == [10, 20, 30, 40] and ring.epoch == 0
    assert lib.libra_ring_neighbors(ring, 10) == (40, 20) and lib.libra_ring_neighbors(ring, 40) == (30, 10)
    lib.libra_ring_remove(ring, 30)                     # a dead peer: its neighbours become each other's
    assert list(ring.members[:ring.n_members]) == [10, 20, 40] and ring.epoch == 1
    assert lib.libra_ring_neighbors(ring, 20) == (10, 40) and lib.libra_ring_neighbors(ring, 40) == (20, 10)
    lib.libra_ring_insert(ring, 50, 1)                  # a joiner, at any position: only its two neighbours change
    assert list(ring.members[:ring.n_members]) == [10, 50, 20, 40] and ring.epoch == 2
    assert lib.libra_ring_neighbors(ring, 50) == (10, 20) and lib.libra_ring_neighbors(ring, 40) == (20, 10)
    assert all(m == -1 for m in ring.members[ring.n_members:])
    for bad in (lambda: lib.libra_ring_remove(ring, 30), lambda: lib.libra_ring_insert(ring, 50, 0),
                lambda: lib.libra_ring_insert(ring, 60, 9), lambda: lib.libra_ring_neighbors(ring, 99),
                lambda: lib.libra_ring_init([1, 2, 1]), lambda: lib.libra_ring_init(list(range(65))),
                lambda: lib.libra_ring_schedule(ring, 10, 24, 16), lambda: lib.libra_ring_schedule(ring, 10, 32, 8),
                lambda: lib.libra_ring_schedule(ring, 77, 32, 16)):
        with pytest.raises(lib.LibraError) as e:
            bad()
        assert e.value.status == lib.INVALID_ARGUMENT
    solo = lib.libra_ring_init([7])
    assert lib.libra_ring_neighbors(solo, 7) == (7, 7) and lib.libra_ring_schedule(solo, 7, 160, 16) == []


def run_schedules(lib, ring, vectors, dtype, piece_bytes):
    """Every live member's schedule executed in lock step with NumPy: all sends of a (phase, step) are taken before any
    receive of it is applied (the members run concurrently).  vectors: {id: float32 array}; returns the same dict."""
    ids = list(ring.members[:ring.n_members])
    elem = 4 if dtype == "f32" else 2      # bytes per element on the wire; values are held as float32 here
    bufs = {i: np.array(vectors[i], dtype=np.float32, copy=True) for i in ids}
    sched = {i: lib.libra_ring_schedule(ring, i, len(bufs[i]) * elem, piece_bytes) for i in ids}
    keys = sorted({(op["phase"], op["step"]) for ops in sched.values() for op in ops})
    for key in keys:
        wire = {}
        for i in ids:
            for op in sched[i]:
                if (op["phase"], op["step"]) == key and op["kind"] == lib.RING_OP_SEND:
                    lo, hi = op["offset"] // elem, (op["offset"] + op["bytes"]) // elem
                    wire[(i, op["peer"], op["segment"], op["piece"])] = (op["offset"], op["bytes"], bufs[i][lo:hi].copy())
        used = set()
        for i in ids:
            for op in sched[i]:
                if (op["phase"], op["step"]) != key or op["kind"] == lib.RING_OP_SEND:
                    continue
                k = (op["peer"], i, op["segment"], op["piece"])
                off, nb, data = wire[k]                       # the predecessor sent exactly this piece
                assert (off, nb) == (op["offset"], op["bytes"])
                used.add(k)
                lo, hi = off // elem, (off + nb) // elem
                bufs[i][lo:hi] = R.add_step(bufs[i][lo:hi], data, dtype) if op["kind"] == lib.RING_OP_RECV_REDUCE else data
        assert used == set(wire)                              # nothing was sent that nobody took
    return bufs


@pytest.mark.parametrize("ranks", [2, 3, 4, 5, 8])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_schedules_fit_together_and_give_the_ring_result(lib, ranks, dtype):
    rng = np.random.default_rng(ranks)
    granule = 4 if dtype == "f32" else 8           # elements per 16-byte unit
    ids = [int(x) for x in rng.permutation(100)[:ranks]]
    for n_units, piece in ((ranks, 16), (5 * ranks + 3, 48), (1000, 1 << 20), (ranks - 1, 16), (257, 160)):
        n = n_units * granule
        xs = [rng.standard_normal(n).astype(np.float32) * np.float32(10.0 ** rng.integers(-3, 4)) for _ in ids]
        if dtype == "bf16":
            xs = [R._bf16_round(x) for x in xs]
        ring = lib.libra_ring_init(ids)
        got = run_schedules(lib, ring, dict(zip(ids, xs)), dtype, piece)
        want = R.ring_all_reduce(xs, dtype, granule=granule)
        for pos, i in enumerate(ids):
            assert np.array_equal(got[i].view(np.uint32), want[pos].view(np.uint32)), (ranks, n_units, piece, pos)
        # the records of one member: pieces tile each segment, segments are the oracle's, peers are the neighbours
        bounds = R.chunk_bounds(n, ranks, granule)
        elem = 16 // granule
        for pos, i in enumerate(ids):
            ops = lib.libra_ring_schedule(ring, i, n * elem, piece)
            pred, succ = lib.libra_ring_neighbors(ring, i)
            assert [(o["phase"], o["step"]) for o in ops] == sorted((o["phase"], o["step"]) for o in ops)
            by = {}
            for o in ops:
                assert o["peer"] == (succ if o["kind"] == lib.RING_OP_SEND else pred)
                assert 0 < o["bytes"] <= piece and o["bytes"] % 16 == 0 and o["offset"] % 16 == 0
                by.setdefault((o["kind"], o["phase"], o["step"], o["segment"]), []).append((o["piece"], o["offset"], o["bytes"]))
            for (kind, phase, step, seg), pieces in by.items():
                assert [p[0] for p in pieces] == list(range(len(pieces)))
                assert pieces[0][1] == bounds[seg] * elem and pieces[-1][1] + pieces[-1][2] == bounds[seg + 1] * elem
                assert all(pieces[k][1] + pieces[k][2] == pieces[k + 1][1] for k in range(len(pieces) - 1))
            rs = [(o["step"], o["segment"]) for o in ops if o["kind"] == lib.RING_OP_RECV_REDUCE and o["piece"] == 0]
            want_rs = [(s, (pos - 1 - s) % ranks) for s in range(ranks - 1) if bounds[(pos - 1 - s) % ranks] < bounds[(pos - 1 - s) % ranks + 1]]
            assert rs == want_rs


def test_a_removed_member_is_skipped_by_everyone(lib):
    rng = np.random.default_rng(1)
    ids = [0, 1, 2, 3, 4]
    xs = {i: rng.standard_normal(400).astype(np.float32) for i in ids}
    ring = lib.libra_ring_init(ids)
    lib.libra_ring_remove(ring, 2)
    live = [0, 1, 3, 4]
    for i in live:
        assert all(op["peer"] != 2 for op in lib.libra_ring_schedule(ring, i, 1600, 1 << 20))
    with pytest.raises(lib.LibraError):
        lib.libra_ring_schedule(ring, 2, 1600, 1 << 20)          # the dead member has no schedule
    got = run_schedules(lib, ring, xs, "f32", 1 << 20)
    want = R.ring_all_reduce([xs[i] for i in live], "f32", granule=4)
    for pos, i in enumerate(live):
        assert np.array_equal(got[i], want[pos])


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


WORKER = r"""
import os, sys, json, time, datetime
sys.path.insert(0, sys.argv[1])
import numpy as np, torch
import torch.distributed as dist
from oracle import ring_oracle as R
from paper_2606_03077_b200 import binding as lib
rank, world = int(sys.argv[3]), 3
dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{sys.argv[2]}", rank=rank, world_size=world)
store = dist.TCPStore("127.0.0.1", int(sys.argv[4]), world, rank == 0, timeout=datetime.timedelta(seconds=60))
n = 4 * 301
vec = lambda r, rnd: np.random.default_rng(100 * rnd + r).standard_normal(n).astype(np.float32)

def exchange(ring, x):
    # this rank's records, in order: a send goes out at once (a copy: the range may change later), a receive blocks
    buf = x.copy()
    pending = []
    for op in lib.libra_ring_schedule(ring, rank, n * 4, 1024):
        lo, hi = op["offset"] // 4, (op["offset"] + op["bytes"]) // 4
        if op["kind"] == lib.RING_OP_SEND:
            pending.append(dist.isend(torch.from_numpy(buf[lo:hi].copy()), dst=op["peer"]))
        else:
            t = torch.empty(hi - lo, dtype=torch.float32)
            dist.recv(t, src=op["peer"])
            buf[lo:hi] = R.add_step(buf[lo:hi], t.numpy(), "f32") if op["kind"] == lib.RING_OP_RECV_REDUCE else t.numpy()
    for p in pending:
        p.wait()
    return buf

ring = lib.libra_ring_init([0, 1, 2])
res = {"rank": rank}
for rnd in (1, 2):
    if rank == 2 and rnd == 2:
        break                                       # this replica stops taking part: it never announces round 2
    store.set(f"ready:{rnd}:{rank}", "1")           # the heartbeat of this round
    for m in list(ring.members[:ring.n_members]):
        try:
            store.wait([f"ready:{rnd}:{m}"], datetime.timedelta(seconds=2.0 if rnd == 2 else 30.0))
        except Exception:                           # no heartbeat in time: the control plane takes the member out
            lib.libra_ring_remove(ring, m)
    live = list(ring.members[:ring.n_members])
    got = exchange(ring, vec(rank, rnd))
    want = R.ring_all_reduce([vec(r, rnd) for r in live], "f32", granule=4)
    res[f"round{rnd}"] = {"live": live, "epoch": int(ring.epoch), "exact": bool(np.array_equal(got, want[live.index(rank)]))}
print(json.dumps(res))
store.set(f"done:{rank}", "1")
store.wait([f"done:{r}" for r in range(world)], datetime.timedelta(seconds=60))   # nobody leaves while others still talk
dist.destroy_process_group()
"""


def test_three_ranks_lose_one_and_carry_on(lib, tmp_path):
    port, port2 = _free_port(), _free_port()
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = [subprocess.Popen([sys.executable, str(script), ROOT, str(port), str(r), str(port2)], stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(3)]
    done = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), [e[-1500:] for _, e in done]
    outs = {o["rank"]: o for o in (json.loads(x.strip().splitlines()[-1]) for x, _ in done)}
    for r in range(3):
        assert outs[r]["round1"] == {"live": [0, 1, 2], "epoch": 0, "exact": True}
    for r in (0, 1):
        assert outs[r]["round2"] == {"live": [0, 1], "epoch": 1, "exact": True}
    assert "round2" not in outs[2]
