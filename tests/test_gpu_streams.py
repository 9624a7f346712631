"""How the step behaves under the launch patterns a serving loop uses: two handles working at the same time on two
streams, and a step with a host plan recorded once in a CUDA graph and replayed while q and the cache contents
change underneath (the lengths, and with them the plan, stay)."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu

HQ, HKV, D = 32, 8, 128


class Job:
    """One handle, its inputs on the device and its own workspace."""

    def __init__(self, lib, seed, lens):
        import torch
        self.torch = torch
        dev = torch.device("cuda:0")
        self.lens, self.bt, self.q, self.k, self.v = W.random_case(seed, len(lens), HQ, HKV, D, lens)
        self.h = lib.Handle(HQ, HKV, D, self.k.shape[0], len(lens), self.bt.shape[1])
        self.ws = torch.empty(self.h.workspace_size(), dtype=torch.uint8, device=dev)
        self.dq, self.dk, self.dv, self.dbt = (H.to_dev(x, dev) for x in (self.q, self.k, self.v, self.bt))
        self.dl = torch.from_numpy(self.lens.copy()).to(dev)
        self.out = torch.full((len(lens), HQ, D), H.CANARY, dtype=torch.int16, device=dev)

    def enqueue(self, stream):
        st = stream.cuda_stream
        self.h.plan(self.lens, self.ws.data_ptr(), self.ws.numel(), st)
        self.h.decode_attn(self.dq.data_ptr(), self.dk.data_ptr(), self.dv.data_ptr(), self.dbt.data_ptr(),
                           self.dl.data_ptr(), self.out.data_ptr(), st)

    def result(self):
        assert self.h.debug_error_word() == 0
        return H.bf16_dev_to_f32(self.out)


def test_two_handles_on_two_streams(lib):
    import torch
    rng = np.random.default_rng(21)
    a = Job(lib, 401, [int(x) for x in rng.integers(1, 6000, size=24)] + [70000])   # one split sequence
    b = Job(lib, 402, [int(x) for x in rng.integers(1, 900, size=40)])               # short units, small blocks
    s0 = torch.cuda.current_stream()
    a.enqueue(s0); b.enqueue(s0)
    torch.cuda.synchronize()
    alone = (a.result().copy(), b.result().copy())
    ref_a, _ = O.paged_decode_attention(a.q[-3:], a.k, a.v, a.bt[-3:], a.lens[-3:])
    assert gates.stated_violations(alone[0][-3:], ref_a) == 0 and gates.tight_violations(alone[0][-3:], ref_a) == 0

    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    for rep in range(20):
        a.out.fill_(H.CANARY); b.out.fill_(H.CANARY)
        torch.cuda.synchronize()
        for _ in range(3):            # both streams hold several steps at once
            a.enqueue(sa); b.enqueue(sb)
        torch.cuda.synchronize()
        assert np.array_equal(a.result(), alone[0]) and np.array_equal(b.result(), alone[1]), rep
    a.h.close(); b.h.close()


@pytest.mark.parametrize("fused", [0, 1])
def test_host_plan_step_replayed_from_a_graph(lib, fused):
    import torch
    dev = torch.device("cuda:0")
    lens = [3000, 17, 0, 1025, 40000, 1]
    j = Job(lib, 403, lens)
    j.h.set_combine_mode(fused)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        j.enqueue(side)               # eager: the first plan into this workspace clears its counters
    side.synchronize()
    eager = j.result().copy()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        st = torch.cuda.current_stream().cuda_stream
        j.h.decode_attn(j.dq.data_ptr(), j.dk.data_ptr(), j.dv.data_ptr(), j.dbt.data_ptr(), j.dl.data_ptr(),
                        j.out.data_ptr(), st)
    j.out.fill_(H.CANARY)
    g.replay(); torch.cuda.synchronize()
    assert np.array_equal(j.result(), eager)

    # new q and new cache contents in the same buffers: the replay sees them
    rng = np.random.default_rng(9)
    q2 = W.f32_to_bf16_bits(rng.standard_normal(j.q.shape, dtype=np.float32))
    k2 = W.f32_to_bf16_bits(rng.standard_normal(j.k.shape, dtype=np.float32))
    v2 = W.f32_to_bf16_bits(rng.standard_normal(j.v.shape, dtype=np.float32))
    j.dq.copy_(H.to_dev(q2, dev)); j.dk.copy_(H.to_dev(k2, dev)); j.dv.copy_(H.to_dev(v2, dev))
    j.out.fill_(H.CANARY)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    got = j.result()
    ref, _ = O.paged_decode_attention(q2, k2, v2, j.bt, j.lens)
    assert np.all(np.isfinite(got))
    assert gates.stated_violations(got, ref) == 0 and gates.tight_violations(got, ref) == 0
    del g
    j.h.close()
