"""GPU parity: the CUDA library, called through its C ABI, against the float64 CPU oracle on the
same seeded inputs.  Gates: the stated one (|err| <= 1e-2 + 1e-2 |ref|) and the tight one
(tests/gates.py).  Integer work (plan, page indexing) is checked bit-exactly."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from oracle import planner_ref as P
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu


def bits(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def check(got, ref, what=""):
    assert np.all(np.isfinite(got)), f"{what}: non-finite output (unwritten row?)"
    assert gates.stated_violations(got, ref) == 0, f"{what}: stated gate"
    assert gates.tight_violations(got, ref) == 0, f"{what}: tight gate, ratio {gates.tight_ratio(got, ref):.2f}"


def small_plan(lib):
    """Planner constants that force splits at test sizes."""
    return lib.PlanParams(4, 1, 2, 16, 16, 64)


# ------------------------------------------------------------------ the tiny workload
def test_tiny_workload(lib):
    lay, q, k, v = W.make_host_inputs("tiny")
    ref, _ = O.paged_decode_attention(q, k, v, lay.block_table, lay.seq_lens)
    got = H.run_host_case(lib, q, k, v, lay.block_table, lay.seq_lens)
    check(got, ref, "tiny")
    got2 = H.run_host_case(lib, q, k, v, lay.block_table, lay.seq_lens, plan=small_plan(lib))
    check(got2, ref, "tiny, forced splits")


# ------------------------------------------------------------------ shapes, tails, layouts
CASES = [
    # (Hq, Hkv, d, lens)
    (4, 1, 64, [1, 2, 15, 16, 17, 31, 33]),
    (8, 2, 128, [255, 256, 257, 1, 700]),
    (8, 8, 128, [100, 1000]),                 # G = 1
    (4, 2, 128, [513, 48]),                   # G = 2
    (40, 8, 128, [1200, 77, 2049]),           # G = 5
    (64, 8, 128, [3000, 5]),                  # G = 8
    (24, 2, 64, [900, 130]),                  # G = 12: two head tiles
    (32, 2, 128, [777, 64]),                  # G = 16
    (6, 2, 64, [0, 40, 0, 300]),              # empty sequences
]


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("case", range(len(CASES)))
def test_shapes_and_tails(lib, case, layout):
    Hq, Hkv, d, lens = CASES[case]
    lens_a, bt, q, k, v = W.random_case(100 + case, len(lens), Hq, Hkv, d, lens)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    for plan in (None, small_plan(lib)):
        got = H.run_host_case(lib, q, k, v, bt, lens_a, layout=layout, plan=plan)
        check(got, ref, f"case {case} {layout} plan={'default' if plan is None else 'small'}")
    # step C as its own kernel gives the same bits as step C inside the decode kernel
    two = H.run_host_case(lib, q, k, v, bt, lens_a, layout=layout, plan=small_plan(lib), fused=0)
    one = H.run_host_case(lib, q, k, v, bt, lens_a, layout=layout, plan=small_plan(lib), fused=1)
    assert np.array_equal(two, got) and np.array_equal(one, got)


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("page_size", [32, 64])
def test_larger_pages(lib, page_size, layout):
    # a page of 32 or 64 tokens is read as 2 or 4 tiles of 16; lengths around page and tile boundaries
    lens = [1, 16, 17, page_size - 1, page_size, page_size + 1, 700, 2049, 0]
    lens_a, bt, q, k, v = W.random_case(60 + page_size, len(lens), 8, 2, 128, lens, page_size=page_size)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    for plan in (None, lib.PlanParams(4, 1, 2, 64, 64, 64)):
        got = H.run_host_case(lib, q, k, v, bt, lens_a, layout=layout, plan=plan)
        check(got, ref, f"page {page_size} {layout}")
    with pytest.raises(lib.LibraError):     # chunks must start on page boundaries
        lib.Handle(8, 2, 128, 64, 4, 8, page_size=page_size, plan=lib.PlanParams(4, 1, 2, 16, 16, 64))


def test_every_block_shape_agrees(lib):
    lens = [2500, 300, 17, 4100]
    lens_a, bt, q, k, v = W.random_case(7, 4, 32, 8, 128, lens)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    for variant in [(4, 3), (4, 2), (4, 4), (4, 6), (8, 2), (8, 3), (2, 6), (2, 4), (12, 2), (2, 2), (6, 2)]:
        got = H.run_host_case(lib, q, k, v, bt, lens_a, plan=lib.PlanParams(8, 1, 2, 256, 256, 64), variant=variant)
        check(got, ref, f"variant {variant}")


def test_plan_too_large_for_kernel_parameters(lib):
    # 40 sequences x 32 chunks = 1280 work items: more than travel with a launch, so the plan is uploaded
    lens = [2048] * 40
    lens_a, bt, q, k, v = W.random_case(9, 40, 4, 1, 64, lens)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    prm = lib.PlanParams(148, 2, 4, 16, 16, 64)
    for variant in [(4, 3), (8, 3)]:
        got = H.run_host_case(lib, q, k, v, bt, lens_a, plan=prm, variant=variant)
        check(got, ref, f"uploaded plan, variant {variant}")
    import torch
    h = lib.Handle(4, 1, 64, k.shape[0], 40, bt.shape[1], plan=prm)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device="cuda:0")
    h.plan(lens_a, ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
    assert len(h.plan_export()["items"]) == 1280
    torch.cuda.synchronize()
    h.close()


def test_longest_supported_sequence(lib):
    # the paper's rollout length cap is 40,960 tokens (2,560 pages); split 64 ways and unsplit
    lens_a, bt, q, k, v = W.random_case(10, 2, 8, 2, 128, [40960, 40959])
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    for plan in (lib.PlanParams(148, 2, 64, 256, 512, 64), lib.PlanParams(148, 2, 1, 256, 512, 1)):
        got = H.run_host_case(lib, q, k, v, bt, lens_a, plan=plan)
        check(got, ref, "40960 tokens")


def test_custom_scale(lib):
    lens_a, bt, q, k, v = W.random_case(8, 2, 8, 2, 64, [90, 33])
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a, sm_scale=0.3)
    got = H.run_host_case(lib, q, k, v, bt, lens_a, sm_scale=0.3)
    check(got, ref, "sm_scale 0.3")


# ------------------------------------------------------------------ the oracle's pins, on the GPU
def test_length_one_is_bit_exact(lib):
    lens_a, bt, q, k, v = W.random_case(21, 3, 8, 2, 128, [1, 1, 1])
    got = H.run_host_case(lib, q, k, v, bt, lens_a)
    for b in range(3):
        for h in range(8):
            assert np.array_equal(got[b, h], W.bf16_bits_to_f32(v[bt[b, 0], h // 4, 0]))


def test_identical_value_rows(lib):
    lens_a, bt, q, k, v = W.random_case(22, 2, 8, 2, 128, [1500, 70])
    row = bits(np.linspace(-3, 3, 128))
    v[...] = row
    got = H.run_host_case(lib, q, k, v, bt, lens_a, plan=small_plan(lib))
    want = W.bf16_bits_to_f32(row)
    # sum p = 1 across pages, warps, splits and the combine: at most one bf16 ulp off
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -7 + 1e-30)


def test_zero_query_mean_closed_form(lib):
    L = 1111
    lens_a, bt, q, k, v = W.random_case(23, 1, 4, 1, 64, [L])
    q[...] = 0
    for t in range(L):
        v[bt[0, t // 16], 0, t % 16] = bits([(t + j) % 251 for j in range(64)])
    exact = np.array([sum((t + j) % 251 for t in range(L)) / L for j in range(64)])
    for plan in (None, small_plan(lib)):
        got = H.run_host_case(lib, q, k, v, bt, lens_a, plan=plan)
        # a lost or doubled 16-token page moves the mean by > 1 %; bf16 output rounding is 0.4 %
        assert np.all(np.abs(got[0] - exact) <= exact * 2.0 ** -7)


def test_one_hot_key_sweep_is_bit_exact(lib):
    L, d = 1000, 64
    lens_a, bt, q, k, v = W.random_case(24, 1, 4, 1, d, [L])
    prm = P.PlanParams(4, 1, 2, 16, 16, 64)
    pl = P.plan([L], 1, prm)
    cuts = sorted({it[2] for it in pl.items} | {it[3] - 1 for it in pl.items})
    sweep = sorted(set(cuts + [0, 15, 16, 31, L - 1, L - 2, 500]))
    assert len(pl.items) > 4
    # value rows encode (page id, slot) as small integers, exact in bf16
    for t in range(L):
        pg = int(bt[0, t // 16])
        v[pg, 0, t % 16] = bits([pg % 256, pg // 256, t % 16] + [(t * 7 + j) % 200 for j in range(d - 3)])
    c = 40.0  # c*c/sqrt(64) = 200: all other weights underflow to 0 in fp32
    import torch
    dev = torch.device("cuda:0")
    r = H.Runner(lib, 4, 1, d, k.shape[0], 1, bt.shape[1], plan=small_plan(lib))
    for tstar in sweep:
        k2 = np.zeros_like(k); q2 = np.zeros_like(q)
        q2[0, :, 0] = bits([c])[0]
        k2[bt[0, tstar // 16], 0, tstar % 16, 0] = bits([c])[0]
        if L % 16:
            k2[bt[0, L // 16], 0, L % 16, 0] = bits([4 * c])[0]     # dominant key one past the end: no effect
        out = H.bf16_dev_to_f32(r.run(H.to_dev(q2, dev), H.to_dev(k2, dev), H.to_dev(v, dev), H.to_dev(bt, dev), lens_a))
        want = W.bf16_bits_to_f32(v[bt[0, tstar // 16], 0, tstar % 16])
        for h in range(4):
            assert np.array_equal(out[0, h], want), f"t*={tstar}"


def test_page_placement_is_bit_invariant(lib):
    lens_a, bt, q, k, v = W.random_case(25, 3, 8, 2, 128, [900, 2100, 33])
    a = H.run_host_case(lib, q, k, v, bt, lens_a, plan=small_plan(lib))
    perm = np.random.default_rng(2).permutation(k.shape[0])
    k2 = np.empty_like(k); v2 = np.empty_like(v)
    k2[perm] = k; v2[perm] = v
    bt2 = np.where(bt >= 0, perm[np.maximum(bt, 0)], -1).astype(np.int32)
    b = H.run_host_case(lib, q, k2, v2, bt2, lens_a, plan=small_plan(lib))
    assert np.array_equal(a, b)


@pytest.mark.parametrize("shift", [100.0, -200.0])
def test_large_key_shift_is_safe(lib, shift):
    # scores move by q0*shift/sqrt(d), up to several hundred: exp would overflow without the running max
    lens_a, bt, q, k, v = W.random_case(26, 2, 8, 2, 64, [400, 90])
    kf = W.bf16_bits_to_f32(k).astype(np.float64)
    kf[..., 0] += shift
    k2 = bits(kf)
    ref, _ = O.paged_decode_attention(q, k2, v, bt, lens_a)
    got = H.run_host_case(lib, q, k2, v, bt, lens_a, plan=small_plan(lib))
    check(got, ref, f"shift {shift}")


def test_split_and_unsplit_agree(lib):
    lens_a, bt, q, k, v = W.random_case(27, 2, 32, 8, 128, [5000, 1300])
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    one = H.run_host_case(lib, q, k, v, bt, lens_a, plan=lib.PlanParams(148, 2, 4, 256, 512, 1))
    many = H.run_host_case(lib, q, k, v, bt, lens_a, plan=lib.PlanParams(148, 2, 4, 256, 512, 64))
    check(one, ref, "max_splits 1")
    check(many, ref, "max_splits 64")


def test_nan_garbage_outside_sequences_is_ignored(lib):
    lens_a, bt, q, k, v = W.random_case(28, 3, 8, 2, 128, [37, 1, 530], poison=False)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    owned = np.zeros((k.shape[0], 16), dtype=bool)
    for b, L in enumerate(lens_a):
        for t in range(int(L)):
            owned[bt[b, t // 16], t % 16] = True
    for arr in (k, v):
        arr.transpose(0, 2, 1, 3)[~owned] = 0x7FC0   # NaN
    got = H.run_host_case(lib, q, k, v, bt, lens_a, plan=small_plan(lib))
    check(got, ref, "NaN garbage")


def test_runs_are_bit_reproducible(lib):
    import torch
    dev = torch.device("cuda:0")
    lens_a, bt, q, k, v = W.random_case(29, 4, 32, 8, 128, [3000, 200, 4500, 1])
    a = H.run_host_case(lib, q, k, v, bt, lens_a)
    b = H.run_host_case(lib, q, k, v, bt, lens_a)
    assert np.array_equal(a, b)
    # many launches on one handle: the arrival counters of the in-kernel combine reset themselves
    r = H.Runner(lib, 32, 8, 128, k.shape[0], 4, bt.shape[1], plan=lib.PlanParams(8, 1, 2, 256, 256, 64))
    args = [H.to_dev(x, dev) for x in (q, k, v, bt)]
    first = H.bf16_dev_to_f32(r.run(*args, lens_a))
    for _ in range(20):
        assert np.array_equal(H.bf16_dev_to_f32(r.run(*args, lens_a)), first)
    r.h.close()


# ------------------------------------------------------------------ device-side checks, host-visible errors
def test_error_word_flags_bad_inputs(lib):
    import torch
    dev = torch.device("cuda:0")
    lens_a, bt, q, k, v = W.random_case(30, 2, 8, 2, 128, [100, 40])
    r = H.Runner(lib, 8, 2, 128, k.shape[0], 2, bt.shape[1])
    args = [H.to_dev(x, dev) for x in (q, k, v)]
    r.run(*args, H.to_dev(bt, dev), lens_a)
    assert r.h.debug_error_word() == 0
    # page id outside the pool: the tiled copy reads zeros there (no fault) and the kernel flags it
    bad = bt.copy(); bad[0, 2] = k.shape[0] + 5
    r.run(*args, H.to_dev(bad, dev), lens_a, check=False)
    assert r.h.debug_error_word() & lib.ERR_BAD_PAGE_ID
    # device lengths that differ from the planned ones
    other = torch.tensor([99, 40], dtype=torch.int32, device=dev)
    r.run(*args, H.to_dev(bt, dev), lens_a, lens_dev=other, check=False)
    assert r.h.debug_error_word() & lib.ERR_SEQ_LEN_MISMATCH
    # and a clean run resets the word
    r.run(*args, H.to_dev(bt, dev), lens_a)
    assert r.h.debug_error_word() == 0


def test_bounded_wait_times_out_cleanly(lib):
    """A wait that can never be satisfied ends by itself, is reported in the error word, and the context
    stays usable: the next step computes correct results."""
    import torch
    dev = torch.device("cuda:0")
    lens_a, bt, q, k, v = W.random_case(31, 2, 8, 2, 128, [100, 40])
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    r = H.Runner(lib, 8, 2, 128, k.shape[0], 2, bt.shape[1])
    args = [H.to_dev(x, dev) for x in (q, k, v, bt)]
    r.run(*args, lens_a)
    r.h.debug_wait_selftest(torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert r.h.debug_error_word() == lib.ERR_WAIT_TIMEOUT
    check(H.bf16_dev_to_f32(r.run(*args, lens_a)), ref, "after a timed-out wait")
    r.h.close()


def test_host_side_misuse(lib):
    import torch
    dev = torch.device("cuda:0")
    h = lib.Handle(8, 2, 128, 64, 4, 8)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    with pytest.raises(lib.LibraError) as e:
        h.decode_attn(ws.data_ptr(), ws.data_ptr(), ws.data_ptr(), ws.data_ptr(), ws.data_ptr(), ws.data_ptr(), st)
    assert e.value.status == lib.NOT_PLANNED
    with pytest.raises(lib.LibraError) as e:
        h.plan(np.array([5], np.int32), ws.data_ptr(), 128, st)
    assert e.value.status == lib.WORKSPACE_TOO_SMALL
    with pytest.raises(lib.LibraError) as e:
        h.plan(np.array([5] * 9, np.int32), ws.data_ptr(), ws.numel(), st)       # batch > max_batch
    assert e.value.status == lib.INVALID_ARGUMENT
    with pytest.raises(lib.LibraError) as e:
        h.plan(np.array([8 * 16 + 1], np.int32), ws.data_ptr(), ws.numel(), st)  # longer than the table row
    assert e.value.status == lib.INVALID_ARGUMENT
    with pytest.raises(lib.LibraError) as e:
        h.plan(np.array([5], np.int32), ws.data_ptr() + 4, ws.numel(), st)       # misaligned workspace
    assert e.value.status == lib.INVALID_ARGUMENT
    h.close()


def test_plan_export_matches_reference(lib):
    import torch
    dev = torch.device("cuda:0")
    lay, _ = W.make_layout("lognormal_b64")
    h = lib.Handle(32, 8, 128, lay.pool_pages, 64, lay.block_table.shape[1])
    prm = h.plan_params()
    assert prm.n_sm == torch.cuda.get_device_properties(0).multi_processor_count
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
    h.plan(lay.seq_lens, ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
    got = h.plan_export()
    ref = P.plan(lay.seq_lens, 8, P.PlanParams(prm.n_sm, prm.ctas_per_sm, prm.items_per_slot, prm.chunk_align,
                                               prm.min_chunk, prm.max_splits, refine=1 if prm.refine > 0 else 0))
    assert got["chunk_target"] == ref.chunk_target and [tuple(r) for r in got["items"]] == ref.items
    assert list(got["num_splits"]) == ref.num_splits and list(got["item_offset"]) == ref.item_offset
    assert list(got["combine"]) == ref.combine
    torch.cuda.synchronize()
    h.close()


def test_host_buffer_entry_point(lib):
    import torch
    dev = torch.device("cuda:0")
    lay, q, k, v = W.make_host_inputs("tiny")
    ref, _ = O.paged_decode_attention(q, k, v, lay.block_table, lay.seq_lens)
    h = lib.Handle(4, 1, 64, lay.pool_pages, 4, lay.block_table.shape[1])
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
    stg = torch.empty(h.host_staging_size(4), dtype=torch.uint8, device=dev)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else np.ascontiguousarray(a)).pin_memory()
    hq, hk, hv, hbt, hl = pin(q), pin(k), pin(v), pin(lay.block_table), pin(lay.seq_lens)
    hout = torch.zeros((4, 4, 64), dtype=torch.int16).pin_memory()
    h.decode_attn_host(hq.data_ptr(), hk.data_ptr(), hv.data_ptr(), hbt.data_ptr(), hl.data_ptr(), 4, hout.data_ptr(),
                       stg.data_ptr(), stg.numel(), ws.data_ptr(), ws.numel(), torch.cuda.current_stream().cuda_stream)
    got = hout.view(torch.bfloat16).float().numpy()
    check(got, ref, "host entry point")
    h.close()


def test_workspace_reused_by_someone_else_needs_invalidate(lib):
    """A workspace that was overwritten between two plans (an allocator handed the address to someone else): after
    libra_workspace_invalidate the next plan clears it again and the split sequences merge correctly."""
    import torch
    dev = torch.device("cuda:0")
    lens = [9000, 40, 5000]
    lens_a, bt, q, k, v = W.random_case(56, 3, 8, 2, 128, lens)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    r = H.Runner(lib, 8, 2, 128, k.shape[0], 3, bt.shape[1], plan=lib.PlanParams(8, 1, 2, 256, 256, 64))
    dq, dk, dv, dbt = (H.to_dev(x, dev) for x in (q, k, v, bt))
    first = H.bf16_dev_to_f32(r.run(dq, dk, dv, dbt, lens_a))
    check(first, ref, "first run")
    r.ws.fill_(0x5A)                      # arrival counters and control words now hold garbage
    torch.cuda.synchronize()
    with pytest.raises(lib.LibraError):   # the plan is dropped with the invalidation
        r.h.workspace_invalidate()
        r.h.decode_attn(dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dbt.data_ptr(), dq.data_ptr(), 0)
    again = H.bf16_dev_to_f32(r.run(dq, dk, dv, dbt, lens_a))   # plans (clearing the workspace) and decodes
    assert np.array_equal(again, first)
    r.h.close()


def test_host_io_entry_point_with_resident_cache(lib):
    """q, block table and lengths from pinned host memory, the cache on the device: the bits of the all-device call."""
    import torch
    dev = torch.device("cuda:0")
    lens = [700, 1, 0, 33, 20000]
    lens_a, bt, q, k, v = W.random_case(55, 5, 32, 8, 128, lens)
    base = H.run_host_case(lib, q, k, v, bt, lens_a)
    h = lib.Handle(32, 8, 128, k.shape[0], 8, bt.shape[1])
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
    stg = torch.empty(h.host_io_staging_size(5), dtype=torch.uint8, device=dev)
    dk, dv = H.to_dev(k, dev), H.to_dev(v, dev)
    hq = torch.from_numpy(q.view(np.int16)).pin_memory()
    hbt, hl = torch.from_numpy(bt.copy()).pin_memory(), torch.from_numpy(lens_a.copy()).pin_memory()
    hout = torch.full((5, 32, 128), H.CANARY, dtype=torch.int16).pin_memory()
    st = torch.cuda.current_stream().cuda_stream
    h.decode_attn_host_io(hq.data_ptr(), dk.data_ptr(), dv.data_ptr(), hbt.data_ptr(), hl.data_ptr(), 5, hout.data_ptr(),
                          stg.data_ptr(), stg.numel(), ws.data_ptr(), ws.numel(), st)
    assert np.array_equal(hout.view(torch.bfloat16).float().numpy(), base)
    with pytest.raises(lib.LibraError):     # staging too small
        h.decode_attn_host_io(hq.data_ptr(), dk.data_ptr(), dv.data_ptr(), hbt.data_ptr(), hl.data_ptr(), 5,
                              hout.data_ptr(), stg.data_ptr(), 256, ws.data_ptr(), ws.numel(), st)
    bad = bt.copy(); bad[4, 3] = k.shape[0] + 9     # a page id outside the pool: reported by the call itself
    hbad = torch.from_numpy(bad).pin_memory()
    with pytest.raises(lib.LibraError) as ei:
        h.decode_attn_host_io(hq.data_ptr(), dk.data_ptr(), dv.data_ptr(), hbad.data_ptr(), hl.data_ptr(), 5,
                              hout.data_ptr(), stg.data_ptr(), stg.numel(), ws.data_ptr(), ws.numel(), st)
    assert ei.value.status == lib.DEVICE_FLAGGED
    h.decode_attn_host_io(hq.data_ptr(), dk.data_ptr(), dv.data_ptr(), hbt.data_ptr(), hl.data_ptr(), 5, hout.data_ptr(),
                          stg.data_ptr(), stg.numel(), ws.data_ptr(), ws.numel(), st)     # and the handle works on
    assert np.array_equal(hout.view(torch.bfloat16).float().numpy(), base)
    h.close()


def test_cache_warmup_never_changes_a_result(lib):
    """The L2 warm-up reads the block table, as a hint, while the kernel before the step may still be writing it.
    Steps queued back to back, each behind kernels that rewrite the WHOLE block table (a new page placement every
    step), the lengths' device copy, q and the pools' contents: the same bits with the warm-up on and off, and the
    oracle's values for the last step."""
    import torch
    dev = torch.device("cuda:0")
    lens = [2500, 300, 17, 4100, 1, 16, 33, 900]
    B, Hq, Hkv, d = len(lens), 32, 8, 128
    lens_a, bt, q, k, v = W.random_case(81, B, Hq, Hkv, d, lens, spare_pages=40)
    rng = np.random.default_rng(82)
    steps = 5
    n_pages = k.shape[0]
    perms = [rng.permutation(n_pages) for _ in range(steps)]            # step i: page p of the case lives at perms[i][p]
    bts = [np.where(bt >= 0, perms[i][np.maximum(bt, 0)], -1).astype(np.int32) for i in range(steps)]
    results = {}
    for warm in (True, False):
        r = H.Runner(lib, Hq, Hkv, d, n_pages, B, bt.shape[1])
        r.h.set_cache_warmup(warm)
        k0, v0 = H.to_dev(k, dev), H.to_dev(v, dev)
        kd, vd = torch.zeros_like(k0), torch.zeros_like(v0)
        btd = torch.full(bt.shape, -1, dtype=torch.int32, device=dev)
        dl = torch.zeros(B, dtype=torch.int32, device=dev)
        qd = torch.zeros((B, Hq, d), dtype=torch.int16, device=dev)
        src_bt = [H.to_dev(x, dev) for x in bts]
        src_perm = [torch.from_numpy(x).to(dev) for x in perms]
        src_l, src_q = torch.from_numpy(lens_a.copy()).to(dev), H.to_dev(q, dev)
        outs = [torch.full((B, Hq, d), H.CANARY, dtype=torch.int16, device=dev) for _ in range(steps)]
        st = torch.cuda.current_stream().cuda_stream
        torch.cuda.synchronize()
        for i in range(steps):      # nothing synchronises inside this loop: the step overlaps the tail of the writers
            kd.index_copy_(0, src_perm[i], k0)
            vd.index_copy_(0, src_perm[i], v0)
            qd.copy_(src_q)
            torch.add(src_l, 0, out=dl)
            torch.add(src_bt[i], 0, out=btd)    # an elementwise KERNEL right before the step writes the block table
            r.h.plan(lens_a, r.ws.data_ptr(), r.ws.numel(), st)
            r.h.decode_attn(qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), dl.data_ptr(), outs[i].data_ptr(), st)
        torch.cuda.synchronize()
        assert r.h.debug_error_word() == 0
        results[warm] = [H.bf16_dev_to_f32(o) for o in outs]
        r.h.close()
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    for i in range(steps):
        assert np.array_equal(results[True][i], results[False][i]), i
        assert np.array_equal(results[True][i], results[True][0]), i      # the placement never changes a result
    check(results[True][-1], ref, "behind writers of the block table")


def test_early_prefetch_is_bit_identical_behind_a_cache_write_kernel(lib):
    """Steps issued back to back, each preceded by kernels that write q and the newest token's K/V rows (what the
    promise of libra_set_early_prefetch allows the preceding kernel to do): same bits as the default."""
    import torch
    dev = torch.device("cuda:0")
    lens = [2500, 300, 17, 4100, 1, 16, 33]
    B, Hq, Hkv, d = len(lens), 32, 8, 128
    lens_a, bt, q, k, v = W.random_case(71, B, Hq, Hkv, d, lens)
    rng = np.random.default_rng(72)
    steps = 4
    new_k = [bits(rng.standard_normal((B, Hkv, d)).astype(np.float32)) for _ in range(steps)]
    new_v = [bits(rng.standard_normal((B, Hkv, d)).astype(np.float32)) for _ in range(steps)]
    new_q = [bits(rng.standard_normal((B, Hq, d)).astype(np.float32)) for _ in range(steps)]
    pages = torch.tensor([bt[b, (lens_a[b] - 1) // 16] for b in range(B)], dtype=torch.long, device=dev)
    slots = torch.tensor([(lens_a[b] - 1) % 16 for b in range(B)], dtype=torch.long, device=dev)
    results = {}
    for early in (False, True):
        r = H.Runner(lib, Hq, Hkv, d, k.shape[0], B, bt.shape[1], plan=lib.PlanParams(148, 1, 1, 256, 512, 64))
        r.h.set_early_prefetch(early)
        kd, vd, btd = H.to_dev(k, dev), H.to_dev(v, dev), H.to_dev(bt, dev)
        qd = torch.zeros((B, Hq, d), dtype=torch.int16, device=dev)
        lens_dev = torch.from_numpy(lens_a).to(dev)
        nk = [H.to_dev(x, dev) for x in new_k]
        nv = [H.to_dev(x, dev) for x in new_v]
        nq = [H.to_dev(x, dev) for x in new_q]
        outs = [torch.zeros((B, Hq, d), dtype=torch.int16, device=dev) for _ in range(steps)]
        st = torch.cuda.current_stream().cuda_stream
        torch.cuda.synchronize()
        for i in range(steps):            # no synchronisation inside: the kernels queue up behind each other
            kd[pages, :, slots, :] = nk[i]        # index_put kernels: the newest token's rows
            vd[pages, :, slots, :] = nv[i]
            qd.copy_(nq[i])                       # a device-to-device copy kernel
            r.h.plan(lens_a, r.ws.data_ptr(), r.ws.numel(), st)
            r.h.decode_attn(qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(),
                            outs[i].data_ptr(), st)
        torch.cuda.synchronize()
        assert r.h.debug_error_word() == 0
        results[early] = [H.bf16_dev_to_f32(o) for o in outs]
        r.h.close()
    for i in range(steps):
        assert np.array_equal(results[True][i], results[False][i]), f"step {i}"
    # and the last step against the oracle on the final pools
    kk, vv = k.copy(), v.copy()
    for b in range(B):
        kk[bt[b, (lens_a[b] - 1) // 16], :, (lens_a[b] - 1) % 16] = new_k[-1][b]
        vv[bt[b, (lens_a[b] - 1) // 16], :, (lens_a[b] - 1) % 16] = new_v[-1][b]
    ref, _ = O.paged_decode_attention(new_q[-1], kk, vv, bt, lens_a)
    check(results[True][-1], ref, "early prefetch, last step")


def test_block_shape_follows_the_longest_unit(lib):
    """Left to itself the library runs a host plan whose units are all short on a small block shape (4 warps x 2
    stages, three blocks per SM; 2 x 2, seven per SM, when none exceeds 256 tokens) and everything else on the default
    one: same bits as asking for that shape."""
    tiny = [1, 100, 256, 16, 0, 33]
    short = [1, 100, 333, 1024, 16, 700, 0, 512]
    mixed = short + [40000]          # the base chunk length grows with the total: units of over 2000 tokens
    for lens, shape in ((tiny, (2, 2)), (short, (4, 2)), (mixed, (8, 3))):
        lens_a, bt, q, k, v = W.random_case(111, len(lens), 32, 8, 128, lens)
        ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
        auto = H.run_host_case(lib, q, k, v, bt, lens_a)
        check(auto, ref, f"auto shape, longest {max(lens)}")
        for variant in ((2, 2), (4, 2), (8, 3)):
            forced = H.run_host_case(lib, q, k, v, bt, lens_a, variant=variant)
            check(forced, ref, f"variant {variant}")
            if variant == shape:
                assert np.array_equal(forced, auto)
