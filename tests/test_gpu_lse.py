"""The optional LSE output (libra_set_lse_output) against the oracle's lse, and what it is for: attention over two
disjoint parts of a sequence, computed as separate rows of one batch, merged with the log-sum-exp rule."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu

LSE_TOL = 4e-3   # P is rounded to bf16 (2^-9 relative per term) before it is summed; lg2 is the approximate instruction


def run_with_lse(lib, q, k, v, bt, lens, plan=None, fused=None, q_len=1, fp8=None):
    import torch
    dev = torch.device("cuda:0")
    B, Hq, d = q.shape[0], q.shape[-2], q.shape[-1]
    Hkv = k.shape[1]
    h = lib.Handle(Hq, Hkv, d, k.shape[0], max(B, 1), bt.shape[1], plan=plan)
    if fp8 is not None:
        h.set_kv_dtype(lib.KV_E4M3, *fp8)
    if fused is not None:
        h.set_combine_mode(fused)
    if q_len > 1:
        h.set_max_query_tokens(q_len)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
    qd, btd = H.to_dev(q, dev), H.to_dev(bt, dev)
    kd = torch.from_numpy(k).to(dev) if fp8 is not None else H.to_dev(k, dev)
    vd = torch.from_numpy(v).to(dev) if fp8 is not None else H.to_dev(v, dev)
    lens_dev = torch.from_numpy(np.ascontiguousarray(lens, dtype=np.int32)).to(dev)
    out = torch.full(q.shape, H.CANARY, dtype=torch.int16, device=dev)
    lse = torch.full(q.shape[:-1], float("nan"), dtype=torch.float32, device=dev)
    h.set_lse_output(lse.data_ptr())
    st = torch.cuda.current_stream().cuda_stream
    h.plan(np.asarray(lens, dtype=np.int32), ws.data_ptr(), ws.numel(), st)
    if q_len > 1:
        h.decode_attn_multi(qd.data_ptr(), q_len, kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(),
                            out.data_ptr(), st)
    else:
        h.decode_attn(qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(), out.data_ptr(), st)
    torch.cuda.synchronize()
    assert h.debug_error_word() == 0
    res = H.bf16_dev_to_f32(out), lse.cpu().numpy()
    h.close()
    return res


def check_lse(got, ref, what):
    assert not np.any(np.isnan(got)), f"{what}: unwritten lse"
    inf = np.isneginf(ref)
    assert np.array_equal(np.isneginf(got), inf), f"{what}: -inf rows differ"
    assert np.max(np.abs(got[~inf] - ref[~inf]), initial=0.0) <= LSE_TOL, f"{what}: {np.max(np.abs(got[~inf] - ref[~inf]))}"


@pytest.mark.parametrize("fused", [0, 1])
def test_lse_of_split_unsplit_and_empty_sequences(lib, fused):
    lens = [2500, 300, 17, 0, 4100, 1]
    lens_a, bt, q, k, v = W.random_case(101, len(lens), 16, 4, 128, lens)
    ref, ref_lse = O.paged_decode_attention(q, k, v, bt, lens_a)
    for plan in (None, lib.PlanParams(8, 1, 2, 256, 256, 64), lib.PlanParams(4, 1, 2, 16, 16, 64)):
        out, lse = run_with_lse(lib, q, k, v, bt, lens_a, plan=plan, fused=fused)
        assert gates.stated_violations(out, ref) == 0 and gates.tight_violations(out, ref) == 0
        check_lse(lse, ref_lse, f"fused={fused}")


def test_lse_with_several_query_tokens_and_with_an_8bit_cache(lib):
    Tq = 3
    lens = [2, 40, 700, 0, 1030]
    lens_a, bt, _, k, v = W.random_case(102, len(lens), 8, 2, 128, lens)
    rng = np.random.default_rng(103)
    q = W.f32_to_bf16_bits(rng.standard_normal((len(lens), Tq, 8, 128)).astype(np.float32))
    ref, ref_lse = O.paged_multi_token_attention(q, k, v, bt, lens_a)
    for plan in (None, lib.PlanParams(4, 1, 2, 16, 16, 64)):
        out, lse = run_with_lse(lib, q, k, v, bt, lens_a, plan=plan, q_len=Tq)
        assert gates.stated_violations(out, ref) == 0 and gates.tight_violations(out, ref) == 0
        check_lse(lse, ref_lse, "multi")
    lens8, bt8, q8, k8, v8 = W.random_case_e4m3(104, 4, 8, 2, 128, [900, 16, 0, 2049])
    ref, ref_lse = O.paged_decode_attention_fp8(q8, k8, v8, bt8, lens8, 0.5, 2.0)
    for plan in (None, lib.PlanParams(4, 1, 2, 16, 16, 64)):
        out, lse = run_with_lse(lib, q8, k8, v8, bt8, lens8, plan=plan, fp8=(0.5, 2.0))
        assert gates.stated_violations(out, ref) == 0 and gates.tight_violations(out, ref) == 0
        check_lse(lse, ref_lse, "8-bit")


def test_two_parts_of_a_sequence_merge_to_the_whole(lib):
    # every sequence is cut at a page boundary into a head part and a tail part, each a row of one batch of 2B
    # "sequences" (the tail's block-table row starts at its first page); out and lse of the two rows merged with
    # the log-sum-exp rule give the attention over the whole sequence
    lens = [700, 33, 2049, 4000]
    B = len(lens)
    lens_a, bt, q, k, v = W.random_case(105, B, 8, 2, 128, lens)
    ref, ref_lse = O.paged_decode_attention(q, k, v, bt, lens_a)
    cut_pages = [(int(L) // 16) // 2 for L in lens_a]           # head part: that many whole pages (may be 0 tokens)
    ld = bt.shape[1]
    bt2 = np.full((2 * B, ld), -1, dtype=np.int32)
    lens2 = np.zeros(2 * B, dtype=np.int32)
    for b in range(B):
        n_pages = (int(lens_a[b]) + 15) // 16
        bt2[2 * b, :cut_pages[b]] = bt[b, :cut_pages[b]]
        lens2[2 * b] = cut_pages[b] * 16
        bt2[2 * b + 1, :n_pages - cut_pages[b]] = bt[b, cut_pages[b]:n_pages]
        lens2[2 * b + 1] = int(lens_a[b]) - cut_pages[b] * 16
    q2 = np.repeat(q, 2, axis=0)
    out, lse = run_with_lse(lib, q2, k, v, bt2, lens2)
    merged = np.zeros_like(ref)
    merged_lse = np.zeros_like(ref_lse)
    for b in range(B):
        for h in range(q.shape[1]):
            o, l = O.merge_partials(out[2 * b:2 * b + 2, h].astype(np.float64), lse[2 * b:2 * b + 2, h].astype(np.float64))
            merged[b, h], merged_lse[b, h] = o, l
    assert gates.stated_violations(merged, ref) == 0
    assert gates.tight_violations(merged, ref) == 0, gates.tight_ratio(merged, ref)   # each part was rounded to bf16 once
    assert np.max(np.abs(merged_lse - ref_lse)) <= 2 * LSE_TOL


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("n_parts", [1, 2, 5, 33, 64])
def test_device_merge_against_the_oracle_merge(lib, n_parts, d):
    """libra_merge_parts on random (out, lse) pairs, some parts empty (lse = -inf, NaN in their out rows), one row
    empty in every part, against the float64 merge of the same bf16 / float32 inputs."""
    import torch
    dev = torch.device("cuda:0")
    rows = 37
    rng = np.random.default_rng(1000 * n_parts + d)
    outs = W.f32_to_bf16_bits(rng.standard_normal((n_parts, rows, d), dtype=np.float32))
    lses = (rng.standard_normal((n_parts, rows)) * 6.0).astype(np.float32)
    empty = rng.random((n_parts, rows)) < 0.2
    empty[:, 5] = True
    if n_parts > 1:
        empty[0, 7] = False
        empty[1:, 7] = True          # exactly one part holds tokens: its row comes back unchanged
    lses[empty] = -np.inf
    outs[empty] = 0x7FC0             # NaN where a part holds nothing
    d_outs, d_lses = H.to_dev(outs, dev), torch.from_numpy(lses).to(dev)
    got = torch.full((rows, d), H.CANARY, dtype=torch.int16, device=dev)
    got_lse = torch.full((rows,), float("nan"), dtype=torch.float32, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    lib.libra_merge_parts(0, d_outs.data_ptr(), d_lses.data_ptr(), n_parts, rows, d, got.data_ptr(), got_lse.data_ptr(), st)
    torch.cuda.synchronize()
    got, got_lse = H.bf16_dev_to_f32(got).astype(np.float64), got_lse.cpu().numpy().astype(np.float64)
    vals = np.where(empty[:, :, None], 0.0, W.bf16_bits_to_f32(outs).astype(np.float64))
    for r in range(rows):
        want, want_lse = O.merge_partials(vals[:, r], lses[:, r].astype(np.float64))
        if np.isneginf(want_lse):
            assert np.isneginf(got_lse[r]) and np.all(got[r] == 0.0)
            continue
        assert np.all(np.abs(got[r] - want) <= 2.0 ** -8 * np.abs(want) + 3e-5), (r, np.max(np.abs(got[r] - want)))
        assert abs(got_lse[r] - want_lse) <= 1e-5 * (1.0 + abs(want_lse)), (r, got_lse[r], want_lse)
    if n_parts > 1:
        assert np.array_equal(got[7], W.bf16_bits_to_f32(outs[0, 7]).astype(np.float64))
    # the second output is optional
    got2 = torch.full((rows, d), H.CANARY, dtype=torch.int16, device=dev)
    lib.libra_merge_parts(0, d_outs.data_ptr(), d_lses.data_ptr(), n_parts, rows, d, got2.data_ptr(), 0, st)
    torch.cuda.synchronize()
    assert np.array_equal(H.bf16_dev_to_f32(got2).astype(np.float64), got)


def test_merge_misuse_is_rejected(lib):
    import torch
    dev = torch.device("cuda:0")
    a = torch.zeros((2, 4, 128), dtype=torch.int16, device=dev)
    l = torch.zeros((2, 4), dtype=torch.float32, device=dev)
    o = torch.zeros((4, 128), dtype=torch.int16, device=dev)
    for args in ((0, a.data_ptr(), l.data_ptr(), 0, 4, 128, o.data_ptr(), 0, 0),
                 (0, a.data_ptr(), l.data_ptr(), 65, 4, 128, o.data_ptr(), 0, 0),
                 (0, a.data_ptr(), l.data_ptr(), 2, 4, 96, o.data_ptr(), 0, 0),
                 (0, a.data_ptr() + 2, l.data_ptr(), 2, 4, 128, o.data_ptr(), 0, 0),
                 (0, 0, l.data_ptr(), 2, 4, 128, o.data_ptr(), 0, 0),
                 (0, a.data_ptr(), l.data_ptr(), 2, -1, 128, o.data_ptr(), 0, 0)):
        with pytest.raises(lib.LibraError):
            lib.libra_merge_parts(*args)
    lib.libra_merge_parts(0, a.data_ptr(), l.data_ptr(), 2, 0, 128, o.data_ptr(), 0, 0)   # no rows: nothing to do


@pytest.mark.parametrize("n_parts", [2, 3, 8])
def test_token_sharded_sequences_merge_on_the_device(lib, n_parts):
    """Every sequence cut at page boundaries into n_parts runs of pages (some empty), the parts decoded as rows of one
    batch laid out part-major - which is the [n_parts][rows][d] layout the merge takes - and merged on the device:
    the attention over the whole sequence."""
    import torch
    dev = torch.device("cuda:0")
    lens = [700, 33, 2049, 4000, 1, 0]
    B, Hq, Hkv, d = len(lens), 8, 2, 128
    lens_a, bt, q, k, v = W.random_case(106, B, Hq, Hkv, d, lens)
    ref, ref_lse = O.paged_decode_attention(q, k, v, bt, lens_a)
    ld = bt.shape[1]
    bt2 = np.full((n_parts * B, ld), -1, dtype=np.int32)
    lens2 = np.zeros(n_parts * B, dtype=np.int32)
    rng = np.random.default_rng(n_parts)
    for b in range(B):
        n_pages = (int(lens_a[b]) + 15) // 16
        cuts = np.sort(rng.integers(0, n_pages + 1, size=n_parts - 1))
        edges = [0] + [int(c) for c in cuts] + [n_pages]
        for i in range(n_parts):
            p0, p1 = edges[i], edges[i + 1]
            bt2[i * B + b, :p1 - p0] = bt[b, p0:p1]
            lens2[i * B + b] = max(0, min(int(lens_a[b]), p1 * 16) - p0 * 16)
        assert lens2[b::B].sum() == lens_a[b]
    q2 = np.tile(q, (n_parts, 1, 1))
    out, lse = run_with_lse(lib, q2, k, v, bt2, lens2)
    parts_out = H.to_dev(W.f32_to_bf16_bits(out.astype(np.float32)), dev)      # exact: out holds bf16 values
    parts_lse = torch.from_numpy(lse).to(dev)
    got = torch.full((B, Hq, d), H.CANARY, dtype=torch.int16, device=dev)
    got_lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=dev)
    lib.libra_merge_parts(0, parts_out.data_ptr(), parts_lse.data_ptr(), n_parts, B * Hq, d, got.data_ptr(),
                          got_lse.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    merged = H.bf16_dev_to_f32(got)
    assert np.all(np.isfinite(merged))
    assert gates.stated_violations(merged, ref) == 0
    assert gates.tight_violations(merged, ref) == 0, gates.tight_ratio(merged, ref)
    got_lse = got_lse.cpu().numpy()
    inf = np.isneginf(ref_lse)
    assert np.array_equal(np.isneginf(got_lse), inf)
    assert np.max(np.abs(got_lse[~inf] - ref_lse[~inf])) <= 2 * LSE_TOL
