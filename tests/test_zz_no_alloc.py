"""The entry point for callers that cannot allocate device memory (libra_decode_attn_static), through
the C ABI.  Such callers -- a server whose allocator is closed after start-up, a plug-in that must not
trigger the device-wide synchronisation of a cudaMalloc inside a running step loop -- pass only inputs
and the output buffer; the workspace is a fixed 8 MiB region inside the library.  The result must be
the one libra_plan + libra_decode_attn give with a caller-owned workspace, on the first call and on a
second call that finds the region as the first one left it.  This file sorts last so that a failure
here cannot hide another test's result in a stop-at-first-failure run."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_workspace_path(lib):
    import torch
    dev = torch.device("cuda:0")
    lens = [5000, 1300, 0, 37, 2049]
    Hq, Hkv, d = 32, 8, 128
    lens_a, bt, q, k, v = W.random_case(41, len(lens), Hq, Hkv, d, lens)
    plan = lib.PlanParams(0, 1, 4, 256, 512, 64)     # several split sequences: partial results go through the scratch
    r = H.Runner(lib, Hq, Hkv, d, k.shape[0], len(lens), bt.shape[1], plan=plan, fused=0)   # decode + combine kernels
    assert r.h.workspace_size() <= lib.STATIC_SCRATCH_BYTES
    dq, dk, dv, dbt = (H.to_dev(x, dev) for x in (q, k, v, bt))
    want = H.bf16_dev_to_f32(r.run(dq, dk, dv, dbt, lens_a))
    assert len(r.h.plan_export()["combine"]) >= 2

    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)   # the definition itself, not only the other entry point

    dl = torch.from_numpy(lens_a.copy()).to(dev)
    st = torch.cuda.current_stream().cuda_stream
    launches = r.h.launch_count()
    outs = [torch.full((len(lens), Hq, d), H.CANARY, dtype=torch.int16, device=dev) for _ in range(2)]
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(dev)[0]
    for call in range(2):   # the second call runs on whatever the first left in the region
        r.h.decode_attn_static(lens_a, dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(),
                               outs[call].data_ptr(), st)
        torch.cuda.synchronize()
        assert r.h.debug_error_word() == 0
    # what the entry point is for: the device's free memory is what it was before the two calls
    assert torch.cuda.mem_get_info(dev)[0] == free_before
    for call in range(2):
        got = H.bf16_dev_to_f32(outs[call])
        assert np.all(np.isfinite(got)), f"call {call}"
        assert gates.stated_violations(got, ref) == 0, f"call {call}"
        assert gates.tight_violations(got, ref) == 0, f"call {call}"
        assert gates.stated_violations(got, want) == 0, f"call {call}"
        assert gates.tight_violations(got, want) == 0, f"call {call}"
        assert np.array_equal(got, want), f"call {call}: same kernels, same order -> same bits"
    assert r.h.launch_count() == launches + 4   # decode + combine, twice: the GPU did the work
    r.h.close()


def test_two_handles_take_turns_on_the_shared_region(lib):
    """Two handles of different shapes alternate on one stream: each call finds the region as the OTHER handle left it
    (other counters, other partial results) and must still give its own workspace-path bits."""
    import torch
    dev = torch.device("cuda:0")
    st = torch.cuda.current_stream().cuda_stream
    cases = []
    for seed, (Hq, Hkv, d, lens) in enumerate([(32, 8, 128, [5000, 1300, 0, 37, 2049]), (8, 2, 64, [3000, 16, 900, 4100])]):
        lens_a, bt, q, k, v = W.random_case(60 + seed, len(lens), Hq, Hkv, d, lens)
        r = H.Runner(lib, Hq, Hkv, d, k.shape[0], len(lens), bt.shape[1], plan=lib.PlanParams(0, 1, 4, 256, 512, 64))
        dq, dk, dv, dbt = (H.to_dev(x, dev) for x in (q, k, v, bt))
        want = H.bf16_dev_to_f32(r.run(dq, dk, dv, dbt, lens_a))
        assert len(r.h.plan_export()["combine"]) >= 1
        dl = torch.from_numpy(lens_a.copy()).to(dev)
        cases.append((r, lens_a, dq, dk, dv, dbt, dl, want, (len(lens), Hq, d)))
    outs = []
    for turn in range(6):   # no synchronisation between the calls: one stream orders them
        r, lens_a, dq, dk, dv, dbt, dl, want, shape = cases[turn & 1]
        out = torch.full(shape, H.CANARY, dtype=torch.int16, device=dev)
        r.h.decode_attn_static(lens_a, dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(),
                               out.data_ptr(), st)
        outs.append(out)
    torch.cuda.synchronize()
    for turn, out in enumerate(outs):
        assert np.array_equal(H.bf16_dev_to_f32(out), cases[turn & 1][7]), turn
    for c in cases:
        assert c[0].h.debug_error_word() == 0
        c[0].h.close()


def test_a_rejected_call_leaves_the_region_and_the_plan_alone(lib):
    """A call that is refused for a bad argument must not clear the shared region (which may hold another call's error
    word) nor re-plan the handle."""
    import torch
    dev = torch.device("cuda:0")
    lens = [600, 3000]
    lens_a, bt, q, k, v = W.random_case(63, len(lens), 8, 2, 128, lens)
    r = H.Runner(lib, 8, 2, 128, k.shape[0], len(lens), bt.shape[1])
    dq, dk, dv, dbt = (H.to_dev(x, dev) for x in (q, k, v, bt))
    want = H.bf16_dev_to_f32(r.run(dq, dk, dv, dbt, lens_a))
    n_items = len(r.h.plan_export()["items"])
    dl = torch.from_numpy(lens_a.copy()).to(dev)
    st = torch.cuda.current_stream().cuda_stream
    out = torch.zeros((len(lens), 8, 128), dtype=torch.int16, device=dev)
    with pytest.raises(lib.LibraError) as e:   # a null output pointer
        r.h.decode_attn_static(np.array([5, 5], np.int32), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(),
                               dl.data_ptr(), 0, st)
    assert e.value.status == lib.INVALID_ARGUMENT
    assert len(r.h.plan_export()["items"]) == n_items          # the handle still holds the plan of `lens`
    r.h.decode_attn(dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(), out.data_ptr(), st)
    torch.cuda.synchronize()
    assert np.array_equal(H.bf16_dev_to_f32(out), want)
    r.h.close()


def test_static_scratch_rejects_shapes_that_need_more(lib):
    import torch
    h = lib.Handle(64, 8, 128, 64, 4096, 8)   # batch bound 4096: far more partial-result room than 8 MiB
    assert h.workspace_size() > lib.STATIC_SCRATCH_BYTES
    z = torch.zeros(64, dtype=torch.int32, device="cuda:0")
    with pytest.raises(lib.LibraError) as e:
        h.decode_attn_static(np.array([5], np.int32), z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(),
                             z.data_ptr(), z.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert e.value.status == lib.WORKSPACE_TOO_SMALL
    h.close()
