"""GPU parity of libra_decode_attn_multi (several query tokens per sequence, causal over the newly appended
tokens) against the float64 CPU oracle, through the C ABI, with the same two gates as single-token decode."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu


def check(got, ref, what=""):
    assert np.all(np.isfinite(got)), f"{what}: non-finite output (unwritten row?)"
    assert gates.stated_violations(got, ref) == 0, f"{what}: stated gate"
    assert gates.tight_violations(got, ref) == 0, f"{what}: tight gate, ratio {gates.tight_ratio(got, ref):.2f}"


def draw_q(seed, B, Tq, Hq, d):
    rng = np.random.default_rng(seed)
    return W.f32_to_bf16_bits(rng.standard_normal((B, Tq, Hq, d)).astype(np.float32))


def run_multi(lib, q, k, v, bt, lens, layout="HND", plan=None, fused=None, max_q=None, page_size=16):
    """q: uint16 [B, Tq, Hq, d] -> float32 [B, Tq, Hq, d]."""
    import torch
    dev = torch.device("cuda:0")
    B, Tq, Hq, d = q.shape
    Hkv = k.shape[1]
    if layout == "NHD":
        k = np.ascontiguousarray(k.transpose(0, 2, 1, 3))
        v = np.ascontiguousarray(v.transpose(0, 2, 1, 3))
    strides = (page_size * Hkv * d, d, Hkv * d) if layout == "NHD" else (0, 0, 0)
    h = lib.Handle(Hq, Hkv, d, k.shape[0], max(B, 1), bt.shape[1], page_size=page_size, kv_strides=strides, plan=plan)
    if fused is not None:
        h.set_combine_mode(fused)
    h.set_max_query_tokens(max_q or Tq)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
    qd, kd, vd, btd = (H.to_dev(x, dev) for x in (q, k, v, bt))
    lens_dev = torch.from_numpy(np.ascontiguousarray(lens, dtype=np.int32)).to(dev)
    out = torch.full((B, Tq, Hq, d), H.CANARY, dtype=torch.int16, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    h.plan(np.asarray(lens, dtype=np.int32), ws.data_ptr(), ws.numel(), st)
    h.decode_attn_multi(qd.data_ptr(), Tq, kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(),
                        out.data_ptr(), st)
    torch.cuda.synchronize()
    assert h.debug_error_word() == 0
    res = H.bf16_dev_to_f32(out)
    h.close()
    return res


def small_plan(lib):
    return lib.PlanParams(4, 1, 2, 16, 16, 64)


CASES = [
    # (Hq, Hkv, d, Tq, lens)
    (4, 1, 64, 4, [4, 5, 16, 17, 19, 33, 300]),         # G = 4, 16 columns
    (8, 2, 128, 2, [255, 256, 257, 2, 700]),            # G = 4
    (8, 8, 128, 16, [16, 100, 1000, 31]),               # G = 1, 16 query tokens: the limits span two tiles
    (64, 8, 128, 2, [3000, 5, 1025]),                   # G = 8
    (40, 8, 128, 3, [1200, 77, 2049]),                  # G = 5, 15 columns
    (6, 2, 64, 5, [0, 40, 3, 300, 1, 5]),               # empty and shorter-than-Tq sequences
    (4, 2, 128, 8, [513, 48, 520]),                     # G = 2
]


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("case", range(len(CASES)))
def test_shapes_tails_and_causal_limits(lib, case, layout):
    Hq, Hkv, d, Tq, lens = CASES[case]
    lens_a, bt, _, k, v = W.random_case(400 + case, len(lens), Hq, Hkv, d, lens)
    q = draw_q(500 + case, len(lens), Tq, Hq, d)
    ref, _ = O.paged_multi_token_attention(q, k, v, bt, lens_a)
    for plan in (None, small_plan(lib)):
        got = run_multi(lib, q, k, v, bt, lens_a, layout=layout, plan=plan)
        check(got, ref, f"case {case} {layout} plan={'default' if plan is None else 'small'}")
    two = run_multi(lib, q, k, v, bt, lens_a, layout=layout, plan=small_plan(lib), fused=0)
    assert np.array_equal(two, got)     # step C as its own kernel: same bits


def test_one_query_token_equals_single_token_entry_point(lib):
    lens = [2500, 300, 17, 4100, 0]
    lens_a, bt, q, k, v = W.random_case(47, len(lens), 32, 8, 128, lens)
    one = H.run_host_case(lib, q, k, v, bt, lens_a)
    multi = run_multi(lib, q[:, None], k, v, bt, lens_a, max_q=2)
    assert np.array_equal(multi[:, 0], one)


def test_rows_match_single_token_steps_at_shorter_lengths(lib):
    # row i of a q_len = 4 step against a single-token step on the sequence cut to L - 3 + i tokens: same
    # inputs, same tolerance class; the two runs split differently, so compare through the oracle's gates
    Tq = 4
    lens = [1030, 2051, 600]
    lens_a, bt, _, k, v = W.random_case(48, 3, 16, 4, 128, lens)
    q = draw_q(49, 3, Tq, 16, 128)
    got = run_multi(lib, q, k, v, bt, lens_a, plan=lib.PlanParams(8, 1, 2, 256, 256, 64))
    for i in range(Tq):
        ref, _ = O.paged_decode_attention(q[:, i], k, v, bt, lens_a - Tq + 1 + i)
        check(got[:, i], ref, f"row {i}")


def test_last_chunk_shorter_than_the_query_block(lib):
    # chunks of 16 tokens: L = 16 j + 1 leaves a last chunk of ONE token, so the earlier query tokens see nothing
    # of it (their partial result is empty) and are masked inside the second-to-last chunk too
    Tq = 4
    lens = [17, 33, 49, 18, 34]
    lens_a, bt, _, k, v = W.random_case(50, len(lens), 4, 1, 64, lens)
    q = draw_q(51, len(lens), Tq, 4, 64)
    ref, _ = O.paged_multi_token_attention(q, k, v, bt, lens_a)
    for fused in (0, 1):
        got = run_multi(lib, q, k, v, bt, lens_a, plan=lib.PlanParams(64, 1, 8, 16, 16, 64), fused=fused)
        check(got, ref, f"short last chunk, fused={fused}")


def test_one_hot_keys_show_the_exact_causal_limit(lib):
    # dominant keys at token 0 and at each new token: row i is the exact mean of the value rows of token 0 and new
    # tokens 0..i (small integers, so the means of 2..5 rows round to bf16 the same way in any order)
    import math
    Tq, d, L = 4, 64, 70
    c = math.sqrt(200.0 * math.sqrt(d))
    lens_a, bt, _, k, v = W.random_case(52, 1, 2, 1, d, [L])
    rng = np.random.default_rng(53)
    vals = rng.integers(-8, 9, size=(L, d)).astype(np.float32)
    new = list(range(L - Tq, L))
    for t in range(L):
        row = np.zeros(d, dtype=np.float32)
        if t == 0 or t in new:
            row[0] = c
        k[bt[0, t // 16], 0, t % 16] = W.f32_to_bf16_bits(row)
        v[bt[0, t // 16], 0, t % 16] = W.f32_to_bf16_bits(vals[t])
    qrow = np.zeros(d, dtype=np.float32)
    qrow[0] = c
    q = np.broadcast_to(W.f32_to_bf16_bits(qrow), (1, Tq, 2, d)).copy()
    for plan in (None, small_plan(lib)):
        got = run_multi(lib, q, k, v, bt, lens_a, plan=plan)
        for i in range(Tq):
            seen = [0] + new[: i + 1]
            want = O.round_to_bf16(vals[seen].astype(np.float64).mean(axis=0))
            # P = 1 exactly for the dominant keys (equal scores), 0 for the rest; the division by the count is the
            # only rounding before the bf16 store
            assert np.max(np.abs(got[0, i, 0] - want)) <= 2.0 ** -7 * np.max(np.abs(want)), f"row {i}"
            assert np.array_equal(got[0, i, 0], got[0, i, 1])


def test_nan_garbage_and_larger_pages(lib):
    # slots past the end of a sequence hold NaN (the generator's poison); page size 32
    Tq = 3
    lens = [1, 16, 17, 31, 32, 33, 700, 2]
    lens_a, bt, _, k, v = W.random_case(54, len(lens), 8, 2, 128, lens, page_size=32)
    q = draw_q(55, len(lens), Tq, 8, 128)
    ref, _ = O.paged_multi_token_attention(q, k, v, bt, lens_a)
    for layout in ("HND", "NHD"):
        got = run_multi(lib, q, k, v, bt, lens_a, layout=layout, plan=lib.PlanParams(4, 1, 2, 32, 32, 64), page_size=32)
        check(got, ref, f"page 32 {layout}")


def test_misuse_is_rejected(lib):
    import torch
    h = lib.Handle(32, 8, 128, 64, 4, 8)
    with pytest.raises(lib.LibraError):
        h.set_max_query_tokens(0)
    with pytest.raises(lib.LibraError):
        h.set_max_query_tokens(5)          # 5 x G = 20 columns
    size1 = h.workspace_size()
    h.set_max_query_tokens(4)
    assert h.workspace_size() > size1
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device="cuda:0")
    st = torch.cuda.current_stream().cuda_stream
    x = torch.zeros(1 << 16, dtype=torch.int16, device="cuda:0")
    with pytest.raises(lib.LibraError):    # the call above dropped the plan
        h.decode_attn_multi(x.data_ptr(), 2, x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), st)
    h.plan(np.array([5], dtype=np.int32), ws.data_ptr(), ws.numel(), st)
    for bad in (0, 5, -1):
        with pytest.raises(lib.LibraError):
            h.decode_attn_multi(x.data_ptr(), bad, x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), st)
    torch.cuda.synchronize()
    h.close()


@pytest.mark.parametrize("layout", ["HND", "NHD"])
def test_append_of_the_new_tokens_fused_in(lib, layout):
    """libra_decode_attn_multi_append: the rows of the newest q_len tokens arrive with the call, land in their slots
    (across a tile and page boundary where the block straddles one) and the output is the oracle's on the updated
    pools; pools afterwards equal the definition bit for bit."""
    import torch
    dev = torch.device("cuda:0")
    Tq = 4
    lens = [4, 5, 16, 17, 18, 19, 20, 33, 300, 1027, 2, 0, 2050]
    B, Hq, Hkv, d = len(lens), 8, 2, 128
    lens_a, bt, _, k, v = W.random_case(120, B, Hq, Hkv, d, lens, poison=False)
    q = draw_q(121, B, Tq, Hq, d)
    rng = np.random.default_rng(122)
    k_new = W.f32_to_bf16_bits(rng.standard_normal((B, Tq, Hkv, d)).astype(np.float32))
    v_new = W.f32_to_bf16_bits(rng.standard_normal((B, Tq, Hkv, d)).astype(np.float32))
    k_ref, v_ref = k.copy(), v.copy()
    for b, L in enumerate(lens_a):
        for i in range(Tq):
            t = int(L) - Tq + i
            if t >= 0:
                k_ref[bt[b, t // 16], :, t % 16, :] = k_new[b, i]
                v_ref[bt[b, t // 16], :, t % 16, :] = v_new[b, i]
    ref, _ = O.paged_multi_token_attention(q, k_ref, v_ref, bt, lens_a)
    kh, vh, strides = k, v, (0, 0, 0)
    if layout == "NHD":
        kh = np.ascontiguousarray(k.transpose(0, 2, 1, 3))
        vh = np.ascontiguousarray(v.transpose(0, 2, 1, 3))
        strides = (16 * Hkv * d, d, Hkv * d)
    for plan in (None, small_plan(lib)):
        for early in (False, True):
            h = lib.Handle(Hq, Hkv, d, k.shape[0], B, bt.shape[1], kv_strides=strides, plan=plan)
            h.set_max_query_tokens(Tq)
            h.set_early_prefetch(early)
            ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
            qd, kd, vd, btd = (H.to_dev(x, dev) for x in (q, kh, vh, bt))
            knd, vnd = H.to_dev(k_new, dev), H.to_dev(v_new, dev)
            lens_dev = torch.from_numpy(lens_a).to(dev)
            out = torch.full((B, Tq, Hq, d), H.CANARY, dtype=torch.int16, device=dev)
            st = torch.cuda.current_stream().cuda_stream
            h.plan(lens_a, ws.data_ptr(), ws.numel(), st)
            h.decode_attn_multi_append(qd.data_ptr(), Tq, knd.data_ptr(), vnd.data_ptr(), kd.data_ptr(), vd.data_ptr(),
                                       btd.data_ptr(), lens_dev.data_ptr(), out.data_ptr(), st)
            torch.cuda.synchronize()
            assert h.debug_error_word() == 0
            check(H.bf16_dev_to_f32(out), ref, f"multi append {layout} early={early}")
            got_k, got_v = kd.cpu().numpy().view(np.uint16), vd.cpu().numpy().view(np.uint16)
            if layout == "NHD":
                got_k, got_v = got_k.transpose(0, 2, 1, 3), got_v.transpose(0, 2, 1, 3)
            assert np.array_equal(got_k, k_ref) and np.array_equal(got_v, v_ref)
            h.close()


def test_two_column_tiles_plan_for_two_slots_per_sm_by_default(lib):
    """More than 8 rows of q per KV head (16 query heads per KV head, or several query tokens): the planner's default
    is two slots per SM and the step runs two 6-warp blocks per SM (bf16 and E4M3 pools alike).  Outputs against the oracle under the default and under a forced one-slot
    plan (the 12-warp block), on the same handle state a caller would have."""
    import torch
    dev = torch.device("cuda:0")
    lens = [5000, 1300, 257, 16, 1, 0, 2048, 90]
    B, Hkv, d = len(lens), 2, 128
    st = torch.cuda.current_stream().cuda_stream
    for Hq, Tq in ((32, 1), (8, 3), (16, 2)):
        lens_a, bt, _, k, v = W.random_case(900 + Hq + Tq, B, Hq, Hkv, d, lens)
        q = draw_q(901 + Hq, B, Tq, Hq, d)
        ref, _ = O.paged_multi_token_attention(q, k, v, bt, lens_a)
        for plan, want in ((None, 2), (lib.PlanParams(0, 1, 0, 0, 0, 0), 1)):
            h = lib.Handle(Hq, Hkv, d, k.shape[0], B, bt.shape[1], plan=plan)
            assert h.plan_params().ctas_per_sm == (want if Hq // Hkv > 8 else 1)
            h.set_max_query_tokens(Tq)
            assert h.plan_params().ctas_per_sm == want
            ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
            qd, kd, vd, btd = (H.to_dev(x, dev) for x in (q, k, v, bt))
            dl = torch.from_numpy(lens_a.copy()).to(dev)
            out = torch.full((B, Tq, Hq, d), H.CANARY, dtype=torch.int16, device=dev)
            h.plan(lens_a, ws.data_ptr(), ws.numel(), st)
            h.decode_attn_multi(qd.data_ptr(), Tq, kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), dl.data_ptr(), out.data_ptr(), st)
            torch.cuda.synchronize()
            assert h.debug_error_word() == 0
            check(H.bf16_dev_to_f32(out), ref, f"Hq {Hq} Tq {Tq} slots {want}")
            # the same plan made on the device: the same bits
            out_d = torch.full((B, Tq, Hq, d), H.CANARY, dtype=torch.int16, device=dev)
            h.plan_device(dl.data_ptr(), B, ws.data_ptr(), ws.numel(), st)
            h.decode_attn_multi(qd.data_ptr(), Tq, kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), dl.data_ptr(), out_d.data_ptr(), st)
            torch.cuda.synchronize()
            assert h.debug_error_word() == 0 and torch.equal(out_d, out)
            h.plan(lens_a, ws.data_ptr(), ws.numel(), st)
            if Tq > 1:   # one query token on the handle laid out for several: the same plan, one column tile
                q1 = np.ascontiguousarray(q[:, :1])
                ref1, _ = O.paged_multi_token_attention(q1, k, v, bt, lens_a)
                out1 = torch.full((B, 1, Hq, d), H.CANARY, dtype=torch.int16, device=dev)
                h.decode_attn(H.to_dev(q1, dev).data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), dl.data_ptr(),
                              out1.data_ptr(), st)
                torch.cuda.synchronize()
                assert h.debug_error_word() == 0
                check(H.bf16_dev_to_f32(out1), ref1, f"Hq {Hq} Tq 1 of {Tq} slots {want}")
            # E4M3 pools plan for two slots by default whatever the rows; here the default is the same under both
            # types, so the plan stays, and the workspace fits either way
            h.set_kv_dtype(lib.KV_E4M3, 1.0, 1.0)
            assert h.plan_params().ctas_per_sm == want and h.workspace_size() <= ws.numel()
            h.set_kv_dtype(lib.KV_BF16)
            h.close()
