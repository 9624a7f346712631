"""GPU parity of the decode step over an E4M3 KV cache (libra_set_kv_dtype) against the float64 CPU oracle,
through the C ABI, with the same two gates as the bf16 cache."""
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


def run_fp8(lib, q, k8, v8, bt, lens, k_scale=1.0, v_scale=1.0, layout="HND", plan=None, fused=None, page_size=16):
    """q: uint16 [B, Hq, d] or [B, Tq, Hq, d]; k8 / v8: uint8 HND pools.  Returns float32 like q."""
    import torch
    dev = torch.device("cuda:0")
    multi = q.ndim == 4
    B, Hq, d = q.shape[0], q.shape[-2], q.shape[-1]
    Tq = q.shape[1] if multi else 1
    Hkv = k8.shape[1]
    strides = (0, 0, 0)
    if layout == "NHD":
        k8 = np.ascontiguousarray(k8.transpose(0, 2, 1, 3))
        v8 = np.ascontiguousarray(v8.transpose(0, 2, 1, 3))
        strides = (page_size * Hkv * d, d, Hkv * d)
    h = lib.Handle(Hq, Hkv, d, k8.shape[0], max(B, 1), bt.shape[1], page_size=page_size, kv_strides=strides, plan=plan)
    h.set_kv_dtype(lib.KV_E4M3, k_scale, v_scale)
    if fused is not None:
        h.set_combine_mode(fused)
    if multi:
        h.set_max_query_tokens(Tq)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
    qd, btd = H.to_dev(q, dev), H.to_dev(bt, dev)
    kd, vd = torch.from_numpy(k8).to(dev), torch.from_numpy(v8).to(dev)
    lens_dev = torch.from_numpy(np.ascontiguousarray(lens, dtype=np.int32)).to(dev)
    out = torch.full(q.shape, H.CANARY, dtype=torch.int16, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    h.plan(np.asarray(lens, dtype=np.int32), ws.data_ptr(), ws.numel(), st)
    if multi:
        h.decode_attn_multi(qd.data_ptr(), Tq, kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(),
                            out.data_ptr(), st)
    else:
        h.decode_attn(qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(), out.data_ptr(), st)
    torch.cuda.synchronize()
    assert h.debug_error_word() == 0
    res = H.bf16_dev_to_f32(out)
    h.close()
    return res


def small_plan(lib):
    return lib.PlanParams(4, 1, 2, 16, 16, 64)


CASES = [
    # (Hq, Hkv, lens)
    (4, 1, [1, 2, 15, 16, 17, 31, 33]),        # G = 4
    (8, 2, [255, 256, 257, 1, 700]),
    (8, 8, [100, 1000]),                       # G = 1
    (40, 8, [1200, 77, 2049]),                 # G = 5
    (64, 8, [3000, 5]),                        # G = 8
    (24, 2, [900, 130]),                       # G = 12: two column tiles
    (32, 2, [777, 64]),                        # G = 16
    (6, 2, [0, 40, 0, 300]),                   # empty sequences
]


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("case", range(len(CASES)))
def test_shapes_and_tails(lib, case, layout):
    Hq, Hkv, lens = CASES[case]
    lens_a, bt, q, k8, v8 = W.random_case_e4m3(600 + case, len(lens), Hq, Hkv, 128, lens)
    ks, vs = 0.75, 1.5
    ref, _ = O.paged_decode_attention_fp8(q, k8, v8, bt, lens_a, ks, vs)
    for plan in (None, small_plan(lib)):
        got = run_fp8(lib, q, k8, v8, bt, lens_a, ks, vs, layout=layout, plan=plan)
        check(got, ref, f"case {case} {layout} plan={'default' if plan is None else 'small'}")
    two = run_fp8(lib, q, k8, v8, bt, lens_a, ks, vs, layout=layout, plan=small_plan(lib), fused=0)
    assert np.array_equal(two, got)


def test_length_one_is_the_scaled_value_row_exactly(lib):
    lens_a, bt, q, k8, v8 = W.random_case_e4m3(620, 3, 8, 2, 128, [1, 1, 1])
    got = run_fp8(lib, q, k8, v8, bt, lens_a, k_scale=3.0, v_scale=0.25)
    for b in range(3):
        for h in range(8):
            want = 0.25 * O.e4m3_to_f64(v8[bt[b, 0], h // 4, 0])      # a power-of-two scale keeps it a bf16 value
            assert np.array_equal(got[b, h].astype(np.float64), want)


def test_every_code_and_every_dim_lands_where_it_should(lib):
    # one-hot keys pick single tokens; their value rows hold the 254 finite codes spread over the 128 dims, so a
    # fragment delivered to the wrong dim, or a code converted wrongly, shows up exactly
    import math
    L, d = 40, 128
    lens_a, bt, _, k8, v8 = W.random_case_e4m3(621, 1, 2, 1, d, [L])
    finite = np.array([c for c in range(256) if c not in (0x7F, 0xFF)], dtype=np.uint8)
    for t in range(L):
        v8[bt[0, t // 16], 0, t % 16] = finite[(np.arange(d) * 2 + 7 * t) % len(finite)]
    # query c e_j against keys 8 e_j at one token: score 8 c k_scale / sqrt(128) >= 150 with c = 256
    for tstar, j in ((0, 0), (15, 1), (16, 2), (17, 3), (31, 64), (39, 127), (22, 77)):
        k8[bt[0], 0] = 0
        k8[bt[0, tstar // 16], 0, tstar % 16, j] = 0x50          # code of 8.0
        qrow = np.zeros(d, dtype=np.float32)
        qrow[j] = 256.0
        q = np.broadcast_to(W.f32_to_bf16_bits(qrow), (1, 2, d)).copy()
        assert 8 * 256 / math.sqrt(d) > 150
        for plan in (None, small_plan(lib)):
            got = run_fp8(lib, q, k8, v8, bt, lens_a, plan=plan)
            want = O.e4m3_to_f64(v8[bt[0, tstar // 16], 0, tstar % 16])
            assert np.array_equal(got[0, 0].astype(np.float64), want), (tstar, j)
            assert np.array_equal(got[0, 1], got[0, 0])


def test_larger_pages(lib):
    lens = [1, 16, 17, 31, 32, 33, 700, 2049, 0]
    lens_a, bt, q, k8, v8 = W.random_case_e4m3(622, len(lens), 8, 2, 128, lens, page_size=32)
    ref, _ = O.paged_decode_attention_fp8(q, k8, v8, bt, lens_a)
    for layout in ("HND", "NHD"):
        for plan in (None, lib.PlanParams(4, 1, 2, 32, 32, 64)):
            got = run_fp8(lib, q, k8, v8, bt, lens_a, layout=layout, plan=plan, page_size=32)
            check(got, ref, f"page 32 {layout}")


def test_several_query_tokens_over_an_8bit_cache(lib):
    # row i of the multi-token step = the single-token definition at length L - Tq + 1 + i
    Tq = 3
    lens = [3, 17, 300, 1030, 2]
    lens_a, bt, _, k8, v8 = W.random_case_e4m3(623, len(lens), 8, 2, 128, lens)
    rng = np.random.default_rng(624)
    q = W.f32_to_bf16_bits(rng.standard_normal((len(lens), Tq, 8, 128)).astype(np.float32))
    for plan in (None, small_plan(lib)):
        got = run_fp8(lib, q, k8, v8, bt, lens_a, 0.5, 2.0, plan=plan)
        for i in range(Tq):
            ref, _ = O.paged_decode_attention_fp8(q[:, i], k8, v8, bt, np.maximum(lens_a - Tq + 1 + i, 0), 0.5, 2.0)
            check(got[:, i], ref, f"row {i}")


def test_split_and_unsplit_agree_and_runs_reproduce(lib):
    lens_a, bt, q, k8, v8 = W.random_case_e4m3(625, 2, 32, 8, 128, [5000, 900])
    ref, _ = O.paged_decode_attention_fp8(q, k8, v8, bt, lens_a)
    one = run_fp8(lib, q, k8, v8, bt, lens_a, plan=lib.PlanParams(148, 1, 1, 256, 512, 1))
    many = run_fp8(lib, q, k8, v8, bt, lens_a, plan=lib.PlanParams(148, 1, 1, 256, 512, 64))
    check(one, ref, "unsplit")
    check(many, ref, "split")
    again = run_fp8(lib, q, k8, v8, bt, lens_a, plan=lib.PlanParams(148, 1, 1, 256, 512, 64))
    assert np.array_equal(again, many)


def test_what_is_not_supported_says_so(lib):
    import torch
    h = lib.Handle(8, 2, 128, 64, 4, 8)
    for bad in ((0.0, 1.0), (1.0, -1.0), (float("inf"), 1.0), (float("nan"), 1.0)):
        with pytest.raises(lib.LibraError):
            h.set_kv_dtype(lib.KV_E4M3, *bad)
    with pytest.raises(lib.LibraError):
        h.set_kv_dtype(7, 1.0, 1.0)
    h.set_kv_dtype(lib.KV_E4M3, 1.0, 1.0)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device="cuda:0")
    st = torch.cuda.current_stream().cuda_stream
    h.plan(np.array([5], dtype=np.int32), ws.data_ptr(), ws.numel(), st)
    x = torch.zeros(1 << 16, dtype=torch.int16, device="cuda:0")
    hs = torch.zeros(1 << 16, dtype=torch.int16).pin_memory()
    with pytest.raises(lib.LibraError):                   # the host-buffer entry point is sized for bf16 pools
        h.decode_attn_host(hs.data_ptr(), hs.data_ptr(), hs.data_ptr(), hs.data_ptr(), hs.data_ptr(), 1, hs.data_ptr(),
                           x.data_ptr(), x.numel() * 2, ws.data_ptr(), ws.numel(), st)
    h.set_kv_dtype(lib.KV_BF16)                           # and back
    torch.cuda.synchronize()
    h.close()
    odd = lib.Handle(8, 2, 128, 64, 4, 8, kv_strides=(16 * 2 * 136, 16 * 136, 136))   # token stride 136: not a multiple of 16
    with pytest.raises(lib.LibraError):
        odd.set_kv_dtype(lib.KV_E4M3, 1.0, 1.0)
    odd.close()


@pytest.mark.parametrize("layout", ["HND", "NHD"])
def test_fused_append_of_8bit_rows(lib, layout):
    # the newest token's K and V rows arrive as E4M3 codes; afterwards the pools hold them and the output is the
    # oracle's on the updated pools
    import torch
    dev = torch.device("cuda:0")
    lens = [1, 16, 17, 300, 1025, 2048, 33]
    B, Hq, Hkv, d = len(lens), 16, 4, 128
    lens_a, bt, q, k8, v8 = W.random_case_e4m3(630, B, Hq, Hkv, d, lens)
    _, _, _, kn, vn = W.random_case_e4m3(631, 1, Hq, Hkv, d, [B], poison=False)     # codes for the new rows
    k_new = np.ascontiguousarray(kn[0, :, :B, :].transpose(1, 0, 2))                 # [B, Hkv, d]
    v_new = np.ascontiguousarray(vn[0, :, :B, :].transpose(1, 0, 2))
    k_ref, v_ref = k8.copy(), v8.copy()
    for b, n in enumerate(lens_a):
        k_ref[bt[b, (n - 1) // 16], :, (n - 1) % 16, :] = k_new[b]
        v_ref[bt[b, (n - 1) // 16], :, (n - 1) % 16, :] = v_new[b]
    ref, _ = O.paged_decode_attention_fp8(q, k_ref, v_ref, bt, lens_a, 0.5, 2.0)
    strides = (0, 0, 0)
    kd_h, vd_h = k8, v8
    if layout == "NHD":
        kd_h = np.ascontiguousarray(k8.transpose(0, 2, 1, 3))
        vd_h = np.ascontiguousarray(v8.transpose(0, 2, 1, 3))
        strides = (16 * Hkv * d, d, Hkv * d)
    for plan in (None, small_plan(lib)):
        h = lib.Handle(Hq, Hkv, d, k8.shape[0], B, bt.shape[1], kv_strides=strides, plan=plan)
        h.set_kv_dtype(lib.KV_E4M3, 0.5, 2.0)
        ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
        qd, btd = H.to_dev(q, dev), H.to_dev(bt, dev)
        kd, vd = torch.from_numpy(kd_h).to(dev), torch.from_numpy(vd_h).to(dev)
        knd, vnd = torch.from_numpy(k_new).to(dev), torch.from_numpy(v_new).to(dev)
        lens_dev = torch.from_numpy(lens_a).to(dev)
        out = torch.full((B, Hq, d), H.CANARY, dtype=torch.int16, device=dev)
        st = torch.cuda.current_stream().cuda_stream
        h.plan(lens_a, ws.data_ptr(), ws.numel(), st)
        h.decode_attn_append(qd.data_ptr(), knd.data_ptr(), vnd.data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(),
                             lens_dev.data_ptr(), out.data_ptr(), st)
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0
        check(H.bf16_dev_to_f32(out), ref, f"append {layout}")
        got_k, got_v = kd.cpu().numpy(), vd.cpu().numpy()
        if layout == "NHD":
            got_k, got_v = got_k.transpose(0, 2, 1, 3), got_v.transpose(0, 2, 1, 3)
        assert np.array_equal(got_k, k_ref) and np.array_equal(got_v, v_ref)
        h.close()


def test_gather_and_scatter_of_8bit_pools(lib):
    # the migration copies on E4M3 pools: gather a head range to a dense buffer, scatter it under a new placement
    import torch
    from oracle import kv_move_oracle as M
    dev = torch.device("cuda:0")
    lens = [40, 1, 16, 333]
    B, Hkv, d, h0, hn = len(lens), 8, 128, 2, 4
    lens_a, bt, _, k8, v8 = W.random_case_e4m3(632, B, Hkv, Hkv, d, lens, poison=False)
    h = lib.Handle(Hkv, Hkv, d, k8.shape[0], B, bt.shape[1])
    h.set_kv_dtype(lib.KV_E4M3, 1.0, 1.0)
    offs = np.concatenate([[0], np.cumsum(lens_a.astype(np.int64))])
    total = int(offs[-1])
    dk, dv, dbt = torch.from_numpy(k8).to(dev), torch.from_numpy(v8).to(dev), H.to_dev(bt, dev)
    dl = torch.from_numpy(lens_a.copy()).to(dev)
    doffs = torch.from_numpy(offs[:-1].copy()).to(dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    k_dense = torch.full((total, hn, d), 0x7F, dtype=torch.uint8, device=dev)
    v_dense = torch.full((total, hn, d), 0x7F, dtype=torch.uint8, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    h.kv_gather(dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(), doffs.data_ptr(), B, int(lens_a.max()),
                h0, hn, k_dense.data_ptr(), v_dense.data_ptr(), err.data_ptr(), st)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    assert np.array_equal(k_dense.cpu().numpy(), M.gather(k8, bt, lens_a, h0, hn))
    assert np.array_equal(v_dense.cpu().numpy(), M.gather(v8, bt, lens_a, h0, hn))
    rng = np.random.default_rng(5)
    bt2, pool2 = W.draw_block_table(lens_a, int(W.pages_needed(lens_a).sum()) + 5, rng, ld=bt.shape[1])
    h2 = lib.Handle(hn, hn, d, pool2, B, bt.shape[1])
    h2.set_kv_dtype(lib.KV_E4M3, 1.0, 1.0)
    k2 = torch.full((pool2, hn, 16, d), 0xEE, dtype=torch.uint8, device=dev)
    v2 = torch.full((pool2, hn, 16, d), 0xEE, dtype=torch.uint8, device=dev)
    dbt2 = H.to_dev(bt2, dev)
    h2.kv_scatter(k_dense.data_ptr(), v_dense.data_ptr(), dbt2.data_ptr(), dl.data_ptr(), doffs.data_ptr(),
                  B, int(lens_a.max()), 0, hn, k2.data_ptr(), v2.data_ptr(), err.data_ptr(), st)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    want_k = np.full((pool2, hn, 16, d), 0xEE, np.uint8)
    want_v = np.full((pool2, hn, 16, d), 0xEE, np.uint8)
    M.scatter(M.gather(k8, bt, lens_a, h0, hn), want_k, bt2, lens_a, 0)
    M.scatter(M.gather(v8, bt, lens_a, h0, hn), want_v, bt2, lens_a, 0)
    assert np.array_equal(k2.cpu().numpy(), want_k) and np.array_equal(v2.cpu().numpy(), want_v)
    h.close(); h2.close()


def test_block_shape_follows_the_longest_unit(lib):
    # batches of short units run on small blocks (several per SM): same bits as asking for that shape, right answers
    import torch
    for lens, shape in (([1, 100, 256, 16, 0, 33], (2, 4)), ([1, 100, 333, 1024, 16, 700, 0, 512], (4, 2))):
        lens_a, bt, q, k8, v8 = W.random_case_e4m3(640, len(lens), 32, 8, 128, lens)
        ref, _ = O.paged_decode_attention_fp8(q, k8, v8, bt, lens_a, 0.5, 2.0)
        auto = run_fp8(lib, q, k8, v8, bt, lens_a, 0.5, 2.0)
        check(auto, ref, f"auto shape, longest {max(lens)}")
        dev = torch.device("cuda:0")
        h = lib.Handle(32, 8, 128, k8.shape[0], len(lens), bt.shape[1])
        h.set_kv_dtype(lib.KV_E4M3, 0.5, 2.0)
        h.set_variant(*shape)
        ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
        qd, btd = H.to_dev(q, dev), H.to_dev(bt, dev)
        kd, vd = torch.from_numpy(k8).to(dev), torch.from_numpy(v8).to(dev)
        lens_dev = torch.from_numpy(lens_a).to(dev)
        out = torch.full(q.shape, H.CANARY, dtype=torch.int16, device=dev)
        st = torch.cuda.current_stream().cuda_stream
        h.plan(lens_a, ws.data_ptr(), ws.numel(), st)
        h.decode_attn(qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(), out.data_ptr(), st)
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0
        assert np.array_equal(H.bf16_dev_to_f32(out), auto)
        h.close()


CASES_D64 = [
    (4, 1, [1, 7, 64, 300]),                   # the tiny workload's shape
    (8, 2, [255, 256, 257, 1, 700, 0]),
    (24, 2, [900, 130, 17]),                   # G = 12: two column tiles
    (8, 8, [100, 1000, 33]),                   # G = 1
]


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("case", range(len(CASES_D64)))
def test_head_dim_64(lib, case, layout):
    # rows of 64 bytes: tiles of 1 KB under the 64-byte swizzle
    Hq, Hkv, lens = CASES_D64[case]
    lens_a, bt, q, k8, v8 = W.random_case_e4m3(650 + case, len(lens), Hq, Hkv, 64, lens)
    ref, _ = O.paged_decode_attention_fp8(q, k8, v8, bt, lens_a, 0.75, 1.5)
    for plan in (None, small_plan(lib)):
        got = run_fp8(lib, q, k8, v8, bt, lens_a, 0.75, 1.5, layout=layout, plan=plan)
        check(got, ref, f"d64 case {case} {layout} plan={'default' if plan is None else 'small'}")


def test_head_dim_64_every_code_and_dim_lands_where_it_should(lib):
    import math
    L, d = 40, 64
    lens_a, bt, _, k8, v8 = W.random_case_e4m3(660, 1, 2, 1, d, [L])
    finite = np.array([c for c in range(256) if c not in (0x7F, 0xFF)], dtype=np.uint8)
    for t in range(L):
        v8[bt[0, t // 16], 0, t % 16] = finite[(np.arange(d) * 3 + 11 * t) % len(finite)]
    for tstar, j in ((0, 0), (15, 1), (16, 2), (17, 31), (31, 32), (39, 63), (22, 47)):
        k8[bt[0], 0] = 0
        k8[bt[0, tstar // 16], 0, tstar % 16, j] = 0x50          # code of 8.0
        qrow = np.zeros(d, dtype=np.float32)
        qrow[j] = 256.0
        q = np.broadcast_to(W.f32_to_bf16_bits(qrow), (1, 2, d)).copy()
        assert 8 * 256 / math.sqrt(d) > 150
        for plan in (None, small_plan(lib)):
            got = run_fp8(lib, q, k8, v8, bt, lens_a, plan=plan)
            want = O.e4m3_to_f64(v8[bt[0, tstar // 16], 0, tstar % 16])
            assert np.array_equal(got[0, 0].astype(np.float64), want), (tstar, j)


def test_head_dim_64_append_and_move(lib):
    import torch
    from oracle import kv_move_oracle as M
    dev = torch.device("cuda:0")
    lens = [1, 16, 17, 300, 33]
    B, Hq, Hkv, d = len(lens), 8, 4, 64
    lens_a, bt, q, k8, v8 = W.random_case_e4m3(670, B, Hq, Hkv, d, lens, poison=False)
    rng = np.random.default_rng(671)
    k_new = rng.integers(0, 0x78, size=(B, Hkv, d)).astype(np.uint8)
    v_new = rng.integers(0, 0x78, size=(B, Hkv, d)).astype(np.uint8)
    k_ref, v_ref = k8.copy(), v8.copy()
    for b, n in enumerate(lens_a):
        k_ref[bt[b, (n - 1) // 16], :, (n - 1) % 16, :] = k_new[b]
        v_ref[bt[b, (n - 1) // 16], :, (n - 1) % 16, :] = v_new[b]
    ref, _ = O.paged_decode_attention_fp8(q, k_ref, v_ref, bt, lens_a)
    h = lib.Handle(Hq, Hkv, d, k8.shape[0], B, bt.shape[1], plan=small_plan(lib))
    h.set_kv_dtype(lib.KV_E4M3, 1.0, 1.0)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
    qd, btd = H.to_dev(q, dev), H.to_dev(bt, dev)
    kd, vd = torch.from_numpy(k8).to(dev), torch.from_numpy(v8).to(dev)
    knd, vnd = torch.from_numpy(k_new).to(dev), torch.from_numpy(v_new).to(dev)
    lens_dev = torch.from_numpy(lens_a).to(dev)
    out = torch.full((B, Hq, d), H.CANARY, dtype=torch.int16, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    h.plan(lens_a, ws.data_ptr(), ws.numel(), st)
    h.decode_attn_append(qd.data_ptr(), knd.data_ptr(), vnd.data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(),
                         lens_dev.data_ptr(), out.data_ptr(), st)
    torch.cuda.synchronize()
    assert h.debug_error_word() == 0
    check(H.bf16_dev_to_f32(out), ref, "d64 append")
    assert np.array_equal(kd.cpu().numpy(), k_ref) and np.array_equal(vd.cpu().numpy(), v_ref)
    # gather heads 1..2 of the updated pools
    offs = np.concatenate([[0], np.cumsum(lens_a.astype(np.int64))])
    doffs = torch.from_numpy(offs[:-1].copy()).to(dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    total = int(offs[-1])
    k_dense = torch.full((total, 2, d), 0x7F, dtype=torch.uint8, device=dev)
    v_dense = torch.full((total, 2, d), 0x7F, dtype=torch.uint8, device=dev)
    h.kv_gather(kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(), doffs.data_ptr(), B, int(lens_a.max()),
                1, 2, k_dense.data_ptr(), v_dense.data_ptr(), err.data_ptr(), st)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    assert np.array_equal(k_dense.cpu().numpy(), M.gather(k_ref, bt, lens_a, 1, 2))
    assert np.array_equal(v_dense.cpu().numpy(), M.gather(v_ref, bt, lens_a, 1, 2))
    h.close()


def test_default_plan_has_two_slots_per_sm_and_switching_the_type_voids_the_plan(lib):
    """Over E4M3 pools the planner's default is two slots per SM (the step runs two blocks per SM), over bf16 pools with
    one column tile it is one: switching the type on a planned handle voids the plan, the workspace still fits, and the
    step planned again is right under either default and under an explicit one-slot plan."""
    import torch
    dev = torch.device("cuda:0")
    lens = [5000, 1300, 257, 16, 1, 0, 2048, 90]
    lens_a, bt, q, k8, v8 = W.random_case_e4m3(660, len(lens), 32, 8, 128, lens)
    ref, _ = O.paged_decode_attention_fp8(q, k8, v8, bt, lens_a, 0.5, 2.0)
    st = torch.cuda.current_stream().cuda_stream
    for plan, want8 in ((None, 2), (lib.PlanParams(0, 1, 0, 0, 0, 0), 1)):
        h = lib.Handle(32, 8, 128, k8.shape[0], len(lens), bt.shape[1], plan=plan)
        assert h.plan_params().ctas_per_sm == 1
        ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
        h.plan(lens_a, ws.data_ptr(), ws.numel(), st)
        h.set_kv_dtype(lib.KV_E4M3, 0.5, 2.0)
        assert h.plan_params().ctas_per_sm == want8 and h.workspace_size() <= ws.numel()
        qd, btd = H.to_dev(q, dev), H.to_dev(bt, dev)
        kd, vd = torch.from_numpy(k8).to(dev), torch.from_numpy(v8).to(dev)
        dl = torch.from_numpy(lens_a.copy()).to(dev)
        out = torch.full(q.shape, H.CANARY, dtype=torch.int16, device=dev)
        args = (qd.data_ptr(), kd.data_ptr(), vd.data_ptr(), btd.data_ptr(), dl.data_ptr(), out.data_ptr(), st)
        if want8 == 2:
            with pytest.raises(lib.LibraError) as e:
                h.decode_attn(*args)
            assert e.value.status == lib.NOT_PLANNED
            h.plan(lens_a, ws.data_ptr(), ws.numel(), st)
        h.decode_attn(*args)
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0
        check(H.bf16_dev_to_f32(out), ref, f"E4M3, {want8} slot(s) per SM")
        h.close()
