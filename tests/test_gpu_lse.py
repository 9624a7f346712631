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
