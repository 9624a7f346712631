"""The device-side planner (libra_plan_device): bit-exact against the reference planner, the decode
step on a device-made plan against the step on a host-made plan, the overflow checks, and a whole step
recorded once in a CUDA graph and replayed over changing lengths."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from oracle import planner_ref as P
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu


def ref_params(h):
    p = h.plan_params()
    return P.PlanParams(p.n_sm, p.ctas_per_sm, p.items_per_slot, p.chunk_align, p.min_chunk, p.max_splits,
                        refine=1 if p.refine > 0 else 0)


def assert_same_plan(got, ref):
    assert got["chunk_target"] == ref.chunk_target
    assert list(got["bucket"]) == ref.bucket
    assert list(got["num_splits"]) == ref.num_splits
    assert list(got["chunk_len"]) == ref.chunk_len
    assert list(got["item_offset"]) == ref.item_offset
    assert [tuple(r) for r in got["items"]] == ref.items
    assert list(got["combine"]) == ref.combine
    assert list(got["empty"]) == ref.empty


def device_plan(lib, lens, hkv, plan=None, ld=None, max_batch=None):
    import torch
    lens = np.asarray(lens, dtype=np.int32)
    B = len(lens)
    ld = ld or max(1, int((lens.max() + 15) // 16) if B else 1)
    h = lib.Handle(hkv * 4, hkv, 128, 16, max_batch or max(B, 1), ld, plan=plan)
    ws = torch.zeros(h.workspace_size(), dtype=torch.uint8, device="cuda:0")
    dl = torch.from_numpy(lens.copy()).to("cuda:0")
    h.plan_device(dl.data_ptr(), B, ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
    return h, ws, dl


@pytest.mark.parametrize("name", W.WORKLOAD_ORDER)
def test_workload_plans_bit_exact(lib, name):
    w = W.WORKLOADS[name]
    for step in range(w.steps):
        lay, _ = W.make_layout(name, step)
        for plan in (None, lib.PlanParams(0, 2, 4, 256, 512, 64)):
            h, ws, dl = device_plan(lib, lay.seq_lens, w.num_kv_heads, plan)
            assert_same_plan(h.plan_export(), P.plan(lay.seq_lens, w.num_kv_heads, ref_params(h)))
            assert h.debug_error_word() == 0
            h.close()


def test_random_and_edge_vectors_bit_exact(lib):
    rng = np.random.default_rng(11)
    cases = [np.zeros(5, np.int32), np.array([1], np.int32), np.array([40960] * 64, np.int32),
             np.array([16, 17, 255, 256, 257, 511, 512, 513, 0, 0, 4096], np.int32),
             np.array([1024] * 7 + [2048] * 3, np.int32)]
    for _ in range(40):
        B = int(rng.integers(1, 600))
        cases.append(np.clip(np.floor(rng.choice([16, 300, 2000, 12000]) * np.exp(rng.normal(size=B) * rng.uniform(0.2, 1.5))),
                             0, 40960).astype(np.int32))
    for i, lens in enumerate(cases):
        hkv = int(rng.choice([1, 2, 8]))
        plan = lib.PlanParams(int(rng.choice([4, 148])), int(rng.integers(1, 4)), int(rng.integers(1, 6)),
                              int(rng.choice([16, 64, 256])), int(rng.choice([16, 512])), int(rng.choice([1, 8, 64])))
        h, ws, dl = device_plan(lib, lens, hkv, plan)
        ref = P.plan(lens, hkv, ref_params(h))
        if len(ref.items) > 4096:
            assert h.debug_error_word() & lib.ERR_PLAN_OVERFLOW
        else:
            assert_same_plan(h.plan_export(), ref)
            assert h.debug_error_word() == 0
        h.close()


def test_large_batches_bit_exact(lib):
    """More items than the planning kernel ranks with its quadratic loop: the sort in shared memory.  Equal lengths
    (every comparison a tie), a few distinct lengths, long-tailed ones; item counts up to the kernel's capacity."""
    rng = np.random.default_rng(13)
    seen = []
    for B in (257, 300, 511, 512, 1000, 2048, 3000, 4096):
        for kind in ("equal", "few", "tail"):
            if kind == "equal":
                lens = np.full(B, int(rng.integers(1, 600)))
            elif kind == "few":
                lens = rng.choice([0, 16, 128, 129, 1024], size=B)
            else:
                lens = np.clip(np.floor(200 * np.exp(rng.normal(size=B) * 1.2)), 0, 40960)
            lens = lens.astype(np.int32)
            hkv = int(rng.choice([1, 8]))
            plan = lib.PlanParams(148, int(rng.choice([1, 7])), int(rng.choice([1, 4])), 16, int(rng.choice([16, 512])), 64)
            h, ws, dl = device_plan(lib, lens, hkv, plan)
            ref = P.plan(lens, hkv, ref_params(h))
            if len(ref.items) > 4096:
                assert h.debug_error_word() & lib.ERR_PLAN_OVERFLOW
            else:
                assert_same_plan(h.plan_export(), ref)
                assert h.debug_error_word() == 0
                seen.append(len(ref.items))
            h.close()
    assert max(seen) > 3000 and sum(n > 400 for n in seen) >= 12
    # a work unit of 2^16 tokens or more among many: the kernel's other sort (its radix sort packs 16-bit lengths)
    for B, long_len, max_splits in ((450, 70000, 1), (1500, 2 ** 20, 8), (4000, 65536, 1)):
        lens = rng.integers(0, 300, B).astype(np.int32)
        lens[rng.integers(0, B)] = long_len
        h, ws, dl = device_plan(lib, lens, 8, lib.PlanParams(148, 1, 1, 16, 16, max_splits))
        ref = P.plan(lens, 8, ref_params(h))
        assert max(e - b for _, _, b, e in ref.items) >= 65536 and 400 < len(ref.items) <= 4096
        assert_same_plan(h.plan_export(), ref)
        assert h.debug_error_word() == 0
        h.close()


def test_few_long_sequences_bit_exact(lib):
    """Small batches of long sequences: plans of fewer than one and a half waves of long blocks, which the planner
    makes again for twice as many slots."""
    import dataclasses
    rng = np.random.default_rng(12)
    refined = 0
    for i in range(120):
        B = int(rng.integers(1, 40))
        base = int(rng.choice([3000, 12000, 20000, 30000]))
        lens = (np.full(B, base) if i % 3 == 0 else
                np.clip(np.floor(base * np.exp(rng.normal(size=B) * rng.uniform(0.05, 0.8))), 0, 40960)).astype(np.int32)
        if i % 5 == 0:
            lens[rng.integers(0, B)] = 0
        hkv = int(rng.choice([1, 2, 4, 8]))
        plan = lib.PlanParams(int(rng.choice([16, 74, 148])), int(rng.integers(1, 3)), int(rng.integers(1, 3)),
                              int(rng.choice([16, 256])), int(rng.choice([16, 512])), int(rng.choice([2, 8, 64])),
                              int(rng.choice([0, 1, -1])))
        h, ws, dl = device_plan(lib, lens, hkv, plan, ld=40960 // 16)
        prm = ref_params(h)
        ref = P.plan(lens, hkv, prm)
        assert_same_plan(h.plan_export(), ref)
        assert h.debug_error_word() == 0
        refined += ref != P.plan(lens, hkv, dataclasses.replace(prm, refine=0))
        h.close()
    assert refined > 3


def test_overflow_is_flagged_and_nothing_runs(lib):
    import torch
    # a length longer than a block-table row can describe
    h, ws, dl = device_plan(lib, [100, 5000], 2, ld=8)
    assert h.debug_error_word() & lib.ERR_PLAN_OVERFLOW
    assert len(h.plan_export()["items"]) == 0
    h.close()
    # more than 4096 work items
    h, ws, dl = device_plan(lib, [40960] * 100, 1, plan=lib.PlanParams(148, 2, 64, 16, 16, 64))
    assert h.debug_error_word() & lib.ERR_PLAN_OVERFLOW
    h.close()
    # more sequences than one block plans
    h = lib.Handle(8, 2, 128, 16, 5000, 4)
    ws = torch.zeros(h.workspace_size(), dtype=torch.uint8, device="cuda:0")
    dl = torch.zeros(5000, dtype=torch.int32, device="cuda:0")
    with pytest.raises(lib.LibraError) as e:
        h.plan_device(dl.data_ptr(), 5000, ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
    assert e.value.status == lib.UNSUPPORTED_SHAPE
    h.close()


def test_step_on_device_plan_equals_step_on_host_plan(lib):
    import torch
    dev = torch.device("cuda:0")
    lens = [5000, 1300, 0, 37, 2049, 1]
    Hq, Hkv, d = 32, 8, 128
    lens_a, bt, q, k, v = W.random_case(51, len(lens), Hq, Hkv, d, lens)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    for plan in (None, lib.PlanParams(0, 2, 8, 256, 256, 64)):
        # same block shape for both (left to itself the library picks a smaller one for a host plan whose units are
        # all short, which a device plan cannot tell it)
        r = H.Runner(lib, Hq, Hkv, d, k.shape[0], len(lens), bt.shape[1], plan=plan, variant=(8, 3))
        dq, dk, dv, dbt = (H.to_dev(x, dev) for x in (q, k, v, bt))
        host = H.bf16_dev_to_f32(r.run(dq, dk, dv, dbt, lens_a))
        dl = torch.from_numpy(lens_a.copy()).to(dev)
        out = torch.full((len(lens), Hq, d), H.CANARY, dtype=torch.int16, device=dev)
        st = torch.cuda.current_stream().cuda_stream
        r.h.plan_device(dl.data_ptr(), len(lens), r.ws.data_ptr(), r.ws.numel(), st)
        r.h.decode_attn(dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(), out.data_ptr(), st)
        torch.cuda.synchronize()
        assert r.h.debug_error_word() == 0
        got = H.bf16_dev_to_f32(out)
        assert np.array_equal(got, host)
        assert gates.tight_violations(got, ref) == 0 and gates.stated_violations(got, ref) == 0
        r.h.close()


def test_recorded_step_replays_over_changing_lengths(lib):
    """plan + decode + combine recorded once in a CUDA graph; every replay plans the lengths that are in
    device memory at that moment."""
    import torch
    dev = torch.device("cuda:0")
    Hq, Hkv, d, B = 16, 4, 128, 6
    steps = [[3000, 40, 1, 700, 2049, 16], [17, 4096, 900, 0, 333, 2500], [1, 1, 1, 1, 1, 1]]
    ld = 4096 // 16
    pool = sum((max(L, 1) + 15) // 16 for L in steps[0]) + 400
    rng = np.random.default_rng(3)
    k = W.f32_to_bf16_bits(rng.standard_normal((pool, Hkv, 16, d), dtype=np.float32))
    v = W.f32_to_bf16_bits(rng.standard_normal((pool, Hkv, 16, d), dtype=np.float32))
    q = W.f32_to_bf16_bits(rng.standard_normal((B, Hq, d), dtype=np.float32))
    h = lib.Handle(Hq, Hkv, d, pool, B, ld, plan=lib.PlanParams(0, 2, 8, 256, 256, 64))
    ws = torch.zeros(h.workspace_size(), dtype=torch.uint8, device=dev)
    dq, dk, dv = (H.to_dev(x, dev) for x in (q, k, v))
    dbt = torch.full((B, ld), -1, dtype=torch.int32, device=dev)
    dl = torch.zeros(B, dtype=torch.int32, device=dev)
    out = torch.zeros((B, Hq, d), dtype=torch.int16, device=dev)

    def tables(lens):
        bt, _ = W.draw_block_table(np.asarray(lens, np.int32), pool, np.random.default_rng(sum(lens)), ld=ld)
        return bt

    side = torch.cuda.Stream()
    bt0 = tables(steps[0])
    dbt.copy_(torch.from_numpy(bt0)); dl.copy_(torch.tensor(steps[0], dtype=torch.int32))
    torch.cuda.synchronize()
    with torch.cuda.stream(side):   # one eager step first: sets up the workspace outside the recording
        h.plan_device(dl.data_ptr(), B, ws.data_ptr(), ws.numel(), side.cuda_stream)
        h.decode_attn(dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(), out.data_ptr(), side.cuda_stream)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        h.plan_device(dl.data_ptr(), B, ws.data_ptr(), ws.numel(), side.cuda_stream)
        h.decode_attn(dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(), out.data_ptr(), side.cuda_stream)
    for lens in steps + [steps[0]]:
        bt = tables(lens)
        dbt.copy_(torch.from_numpy(bt)); dl.copy_(torch.tensor(lens, dtype=torch.int32))
        out.fill_(H.CANARY)
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        got = H.bf16_dev_to_f32(out)
        ref, _ = O.paged_decode_attention(q, k, v, bt, np.asarray(lens, np.int32))
        assert np.all(np.isfinite(got))
        assert gates.tight_violations(got, ref) == 0 and gates.stated_violations(got, ref) == 0, lens
    assert h.debug_error_word() == 0
    h.close()


def test_separate_combine_with_nothing_to_merge_keeps_the_chain_ordered(lib):
    """Device-side plan, step C as its own kernel, and a batch in which no sequence is split: every block of the
    combine grid has nothing to do.  It must still wait for the decode kernel before it ends, or the next step in
    the stream (a programmatic dependent of the combine grid) could overtake a decode kernel that is still writing.
    A chain of such steps that feed each other (each step's q is the previous step's output) gives the bits of the
    chain run with step C inside the decode kernel."""
    import torch
    dev = torch.device("cuda:0")
    lens = [700, 40, 1, 333, 512, 16, 0, 90]
    Hq, Hkv, d = 32, 8, 128
    lens_a, bt, q, k, v = W.random_case(77, len(lens), Hq, Hkv, d, lens)
    dq, dk, dv, dbt = (H.to_dev(x, dev) for x in (q, k, v, bt))
    dl = torch.from_numpy(lens_a.copy()).to(dev)
    results = []
    for mode in (1, 0):
        r = H.Runner(lib, Hq, Hkv, d, k.shape[0], len(lens), bt.shape[1], variant=(8, 3), fused=mode,
                     plan=lib.PlanParams(0, 0, 0, 0, 0, 0, -1))   # the plain plan: every sequence stays in one piece
        st = torch.cuda.current_stream().cuda_stream
        bufs = [dq.clone(), torch.zeros_like(dq)]
        r.h.plan_device(dl.data_ptr(), len(lens), r.ws.data_ptr(), r.ws.numel(), st)
        for i in range(24):   # back to back, no host synchronisation in between
            r.h.decode_attn(bufs[i & 1].data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(),
                            bufs[(i + 1) & 1].data_ptr(), st)
        torch.cuda.synchronize()
        assert r.h.debug_error_word() == 0
        assert len(r.h.plan_export()["combine"]) == 0
        results.append(bufs[0].cpu().numpy().copy())
        r.h.close()
    assert np.array_equal(results[0], results[1])


@pytest.mark.parametrize("L,hint", [(200, 256), (900, 1024), (900, 0), (900, 256)])
def test_length_hint_picks_the_block_shape_of_a_host_plan(lib, L, hint):
    """A device-planned batch of short sequences with the caller's bound on the lengths runs on the block shape a host
    plan would have picked: the same bits as the host-planned step.  Without the hint (or with one that turns out too
    small) the result is as correct, on another shape."""
    import torch
    dev = torch.device("cuda:0")
    B, Hq, Hkv, d = 40, 32, 8, 128
    lens = [L - (i % 7) * 3 for i in range(B)]
    lens_a, bt, q, k, v = W.random_case(130 + L, B, Hq, Hkv, d, lens)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    r = H.Runner(lib, Hq, Hkv, d, k.shape[0], B, bt.shape[1])
    dq, dk, dv, dbt = (H.to_dev(x, dev) for x in (q, k, v, bt))
    host = H.bf16_dev_to_f32(r.run(dq, dk, dv, dbt, lens_a))          # host plan: the library sees the longest unit
    dl = torch.from_numpy(lens_a.copy()).to(dev)
    out = torch.full((B, Hq, d), H.CANARY, dtype=torch.int16, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    r.h.set_length_hint(hint)
    r.h.plan_device(dl.data_ptr(), B, r.ws.data_ptr(), r.ws.numel(), st)
    r.h.decode_attn(dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(), out.data_ptr(), st)
    torch.cuda.synchronize()
    assert r.h.debug_error_word() == 0
    got = H.bf16_dev_to_f32(out)
    assert gates.tight_violations(got, ref) == 0 and gates.stated_violations(got, ref) == 0
    if hint >= L:
        assert np.array_equal(got, host)
    r.h.close()
