"""Write-bounds evidence: every buffer the library writes -- `out`, the workspace, the optional lse output, the dense
buffers of the KV move, the pools of a scatter or a fused append, the output of the part merge, the destination of a
ring step -- is placed inside a larger allocation with a 4 KB band of known bytes directly before and directly after
it.  After each call every band byte must be what it was and the device error word must be 0.  The payload starts
and ends exactly at the band (no rounding of the end), so a write one element past a buffer lands in a band.
Small cases only; each also checks the result, so that a band is never "untouched" because nothing ran."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from oracle import kv_move_oracle as M
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu

BAND = 4096


class Banded:
    """`nbytes` of device memory between two bands; `t` is the payload as a uint8 tensor, `ptr` its address."""

    registry = None   # the list that collects the buffers of one test

    def __init__(self, nbytes, fill=0):
        import torch
        dev = torch.device("cuda:0")
        nbytes = int(nbytes)
        self.raw = torch.empty(BAND + nbytes + BAND, dtype=torch.uint8, device=dev)
        gen = torch.Generator(device=dev).manual_seed(nbytes % 9973 + 5)
        self.before = torch.randint(1, 255, (BAND,), dtype=torch.uint8, device=dev, generator=gen)
        self.after = torch.randint(1, 255, (BAND,), dtype=torch.uint8, device=dev, generator=gen)
        self.raw[:BAND] = self.before
        self.raw[BAND + nbytes:] = self.after
        self.t = self.raw[BAND:BAND + nbytes]
        self.t.fill_(fill)
        self.ptr = self.t.data_ptr()
        assert self.ptr % 256 == 0
        if Banded.registry is not None:
            Banded.registry.append(self)

    @classmethod
    def of(cls, array):
        """A banded device copy of a host array."""
        import torch
        a = np.ascontiguousarray(array)
        b = cls(a.nbytes)
        b.t.copy_(torch.from_numpy(a.view(np.uint8).reshape(-1)))
        return b

    def host(self, dtype, shape):
        return self.t.cpu().numpy().view(dtype).reshape(shape)

    def intact(self):
        import torch
        n = self.t.numel()
        return bool(torch.equal(self.raw[:BAND], self.before)) and bool(torch.equal(self.raw[BAND + n:], self.after))


@pytest.fixture
def bands():
    Banded.registry = []
    yield Banded.registry
    Banded.registry = None


def all_intact(bands):
    import torch
    torch.cuda.synchronize()
    bad = [i for i, b in enumerate(bands) if not b.intact()]
    assert not bad, f"band bytes changed around buffer(s) {bad}"


def bf16(banded, shape):
    return H.bf16_dev_to_f32(banded.t.view(__import__("torch").int16).reshape(shape))


CASES = [(32, 8, 128, [5000, 1300, 0, 37, 2049, 1]), (4, 1, 64, [300, 64, 7, 1]), (40, 8, 128, [48, 1025, 16])]


@pytest.mark.parametrize("Hq,Hkv,d,lens", CASES)
@pytest.mark.parametrize("fused", [1, 0])
@pytest.mark.parametrize("device_plan", [False, True])
def test_decode_stays_inside_out_workspace_and_lse(lib, bands, Hq, Hkv, d, lens, fused, device_plan):
    import torch
    B = len(lens)
    lens_a, bt, q, k, v = W.random_case(81, B, Hq, Hkv, d, lens)
    ref, ref_lse = O.paged_decode_attention(q, k, v, bt, lens_a)
    for plan in (None, lib.PlanParams(4, 1, 2, 16, 16, 64)):     # default (mostly unsplit) and many small chunks
        h = lib.Handle(Hq, Hkv, d, k.shape[0], B, bt.shape[1], plan=plan)
        h.set_combine_mode(fused)
        ws = Banded(h.workspace_size(), fill=0xEE)                # exactly the size the library asks for
        out = Banded(B * Hq * d * 2, fill=0xC0)
        lse = Banded(B * Hq * 4, fill=0xC0)
        dq, dk, dv, dbt, dl = (Banded.of(x) for x in (q, k, v, bt, lens_a))
        h.set_lse_output(lse.ptr)
        st = torch.cuda.current_stream().cuda_stream
        for _ in range(2):   # the second call runs on the workspace as the first left it
            if device_plan:
                h.plan_device(dl.ptr, B, ws.ptr, ws.t.numel(), st)
            else:
                h.plan(lens_a, ws.ptr, ws.t.numel(), st)
            h.decode_attn(dq.ptr, dk.ptr, dv.ptr, dbt.ptr, dl.ptr, out.ptr, st)
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0
        all_intact(bands)
        got = bf16(out, (B, Hq, d))
        assert gates.stated_violations(got, ref) == 0 and gates.tight_violations(got, ref) == 0
        got_lse = lse.host(np.float32, (B, Hq)).astype(np.float64)
        live = np.isfinite(ref_lse)
        assert np.all(np.abs(got_lse[live] - ref_lse[live]) <= 4e-3) and np.all(got_lse[~live] == -np.inf)
        h.close()


def test_static_scratch_entry_stays_inside_out(lib, bands):
    import torch
    Hq, Hkv, d, lens = 32, 8, 128, [5000, 1300, 0, 37, 2049]
    lens_a, bt, q, k, v = W.random_case(82, len(lens), Hq, Hkv, d, lens)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)
    h = lib.Handle(Hq, Hkv, d, k.shape[0], len(lens), bt.shape[1], plan=lib.PlanParams(0, 1, 4, 256, 512, 64))
    out = Banded(len(lens) * Hq * d * 2, fill=0xC0)
    dq, dk, dv, dbt, dl = (Banded.of(x) for x in (q, k, v, bt, lens_a))
    h.decode_attn_static(lens_a, dq.ptr, dk.ptr, dv.ptr, dbt.ptr, dl.ptr, out.ptr, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert h.debug_error_word() == 0
    all_intact(bands)
    got = bf16(out, (len(lens), Hq, d))
    assert gates.stated_violations(got, ref) == 0 and gates.tight_violations(got, ref) == 0
    h.close()


def test_8bit_cache_and_several_query_tokens_stay_inside(lib, bands):
    import torch
    st = torch.cuda.current_stream().cuda_stream
    # E4M3 cache
    Hq, Hkv, d, lens = 32, 8, 128, [3000, 700, 0, 17, 1]
    lens_a, bt, q, k8, v8 = W.random_case_e4m3(83, len(lens), Hq, Hkv, d, lens)
    ref, _ = O.paged_decode_attention_fp8(q, k8, v8, bt, lens_a, 0.5, 1.25)
    for plan in (None, lib.PlanParams(4, 1, 2, 16, 16, 64)):
        h = lib.Handle(Hq, Hkv, d, k8.shape[0], len(lens), bt.shape[1], plan=plan)
        h.set_kv_dtype(lib.KV_E4M3, 0.5, 1.25)
        ws = Banded(h.workspace_size(), fill=0xEE)
        out = Banded(len(lens) * Hq * d * 2, fill=0xC0)
        dq, dk, dv, dbt, dl = (Banded.of(x) for x in (q, k8, v8, bt, lens_a))
        h.plan(lens_a, ws.ptr, ws.t.numel(), st)
        h.decode_attn(dq.ptr, dk.ptr, dv.ptr, dbt.ptr, dl.ptr, out.ptr, st)
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0
        all_intact(bands)
        got = bf16(out, (len(lens), Hq, d))
        assert gates.stated_violations(got, ref) == 0 and gates.tight_violations(got, ref) == 0
        h.close()
    # several query tokens, with and without the fused append of their rows
    Hq, Hkv, d, Tq, lens = 8, 2, 128, 3, [700, 33, 3, 2, 1, 1030]
    B = len(lens)
    lens_a, bt, _, k, v = W.random_case(84, B, Hq, Hkv, d, lens)
    rng = np.random.default_rng(9)
    q = W.f32_to_bf16_bits(rng.standard_normal((B, Tq, Hq, d), dtype=np.float32))
    ref, _ = O.paged_multi_token_attention(q, k, v, bt, lens_a)
    for plan in (None, lib.PlanParams(4, 1, 2, 16, 16, 64)):
        h = lib.Handle(Hq, Hkv, d, k.shape[0], B, bt.shape[1], plan=plan)
        h.set_max_query_tokens(Tq)
        ws = Banded(h.workspace_size(), fill=0xEE)
        out = Banded(B * Tq * Hq * d * 2, fill=0xC0)
        dq, dk, dv, dbt, dl = (Banded.of(x) for x in (q, k, v, bt, lens_a))
        h.plan(lens_a, ws.ptr, ws.t.numel(), st)
        h.decode_attn_multi(dq.ptr, Tq, dk.ptr, dv.ptr, dbt.ptr, dl.ptr, out.ptr, st)
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0
        all_intact(bands)
        got = bf16(out, (B, Tq, Hq, d))
        assert gates.stated_violations(got, ref) == 0 and gates.tight_violations(got, ref) == 0
        h.close()


@pytest.mark.parametrize("Tq", [1, 2])
def test_fused_append_writes_only_its_rows(lib, bands, Tq):
    """The pools themselves sit between bands, and inside the pools only the new tokens' rows may change."""
    import torch
    Hq, Hkv, d, lens = 8, 2, 128, [1, 16, 17, 33, 700, 2]
    B = len(lens)
    lens_a, bt, _, k, v = W.random_case(85, B, Hq, Hkv, d, lens, poison=False)
    rng = np.random.default_rng(10)
    q = W.f32_to_bf16_bits(rng.standard_normal((B, Tq, Hq, d), dtype=np.float32))
    k_new = W.f32_to_bf16_bits(rng.standard_normal((B, Tq, Hkv, d), dtype=np.float32))
    v_new = W.f32_to_bf16_bits(rng.standard_normal((B, Tq, Hkv, d), dtype=np.float32))
    k_ref, v_ref = k.copy(), v.copy()
    for b, L in enumerate(lens):
        for i in range(Tq):
            t = L - Tq + i
            if t >= 0:
                k_ref[bt[b, t // 16], :, t % 16, :] = k_new[b, i]
                v_ref[bt[b, t // 16], :, t % 16, :] = v_new[b, i]
    ref, _ = O.paged_multi_token_attention(q, k_ref, v_ref, bt, lens_a)
    for plan in (None, lib.PlanParams(4, 1, 2, 16, 16, 64)):
        h = lib.Handle(Hq, Hkv, d, k.shape[0], B, bt.shape[1], plan=plan)
        h.set_max_query_tokens(Tq)
        ws = Banded(h.workspace_size(), fill=0xEE)
        out = Banded(B * Tq * Hq * d * 2, fill=0xC0)
        dq, dk, dv, dbt, dl, dkn, dvn = (Banded.of(x) for x in (q, k, v, bt, lens_a, k_new, v_new))
        st = torch.cuda.current_stream().cuda_stream
        h.plan(lens_a, ws.ptr, ws.t.numel(), st)
        if Tq == 1:
            h.decode_attn_append(dq.ptr, dkn.ptr, dvn.ptr, dk.ptr, dv.ptr, dbt.ptr, dl.ptr, out.ptr, st)
        else:
            h.decode_attn_multi_append(dq.ptr, Tq, dkn.ptr, dvn.ptr, dk.ptr, dv.ptr, dbt.ptr, dl.ptr, out.ptr, st)
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0
        all_intact(bands)
        assert np.array_equal(dk.host(np.uint16, k.shape), k_ref) and np.array_equal(dv.host(np.uint16, v.shape), v_ref)
        got = bf16(out, (B, Tq, Hq, d))
        assert gates.stated_violations(got, ref) == 0 and gates.tight_violations(got, ref) == 0
        h.close()


@pytest.mark.parametrize("h0,hn", [(0, 4), (1, 2), (3, 1)])
def test_kv_gather_and_scatter_stay_inside(lib, bands, h0, hn):
    import torch
    Hkv, d, lens = 4, 128, [1, 16, 17, 700, 0, 333]
    B = len(lens)
    lens_a, bt, _, k, v = W.random_case(86, B, Hkv, Hkv, d, lens, poison=False)
    h = lib.Handle(Hkv, Hkv, d, k.shape[0], B, bt.shape[1])
    offs = np.concatenate([[0], np.cumsum(lens_a.astype(np.int64))])
    total = int(offs[-1])
    dk, dv, dbt, dl, doffs = (Banded.of(x) for x in (k, v, bt, lens_a, offs[:-1].astype(np.int64)))
    err = Banded(4)
    kd, vd = Banded(total * hn * d * 2, fill=0xC0), Banded(total * hn * d * 2, fill=0xC0)   # exactly the rows gathered
    st = torch.cuda.current_stream().cuda_stream
    h.kv_gather(dk.ptr, dv.ptr, dbt.ptr, dl.ptr, doffs.ptr, B, int(lens_a.max()), h0, hn, kd.ptr, vd.ptr, err.ptr, st)
    torch.cuda.synchronize()
    assert err.host(np.int32, (1,))[0] == 0
    all_intact(bands)
    assert np.array_equal(kd.host(np.uint16, (total, hn, d)), M.gather(k, bt, lens_a, h0, hn))
    assert np.array_equal(vd.host(np.uint16, (total, hn, d)), M.gather(v, bt, lens_a, h0, hn))
    # scatter the rows back into zeroed pools: only the owned slots of heads [h0, h0 + hn) may change
    k2, v2 = Banded(k.nbytes, fill=0), Banded(v.nbytes, fill=0)
    h.kv_scatter(kd.ptr, vd.ptr, dbt.ptr, dl.ptr, doffs.ptr, B, int(lens_a.max()), h0, hn, k2.ptr, v2.ptr, err.ptr, st)
    torch.cuda.synchronize()
    assert err.host(np.int32, (1,))[0] == 0
    all_intact(bands)
    want_k, want_v = np.zeros_like(k), np.zeros_like(v)
    for b, L in enumerate(lens):
        for t in range(L):
            want_k[bt[b, t // 16], h0:h0 + hn, t % 16] = k[bt[b, t // 16], h0:h0 + hn, t % 16]
            want_v[bt[b, t // 16], h0:h0 + hn, t % 16] = v[bt[b, t // 16], h0:h0 + hn, t % 16]
    assert np.array_equal(k2.host(np.uint16, k.shape), want_k) and np.array_equal(v2.host(np.uint16, v.shape), want_v)
    h.close()


@pytest.mark.parametrize("n_parts,rows,d", [(2, 5, 128), (3, 33, 64), (8, 1, 128)])
def test_part_merge_stays_inside(lib, bands, n_parts, rows, d):
    import torch
    rng = np.random.default_rng(n_parts)
    po = W.f32_to_bf16_bits(rng.standard_normal((n_parts, rows, d), dtype=np.float32))
    pl = rng.standard_normal((n_parts, rows)).astype(np.float32)
    dpo, dpl = Banded.of(po), Banded.of(pl)
    out, lse = Banded(rows * d * 2, fill=0xC0), Banded(rows * 4, fill=0xC0)
    lib.libra_merge_parts(0, dpo.ptr, dpl.ptr, n_parts, rows, d, out.ptr, lse.ptr, torch.cuda.current_stream().cuda_stream)
    all_intact(bands)
    o64 = O.bf16_bits_to_f64(po)
    w = np.exp(pl.astype(np.float64) - pl.max(axis=0))
    want = (w[..., None] * o64).sum(0) / w.sum(0)[..., None]
    got = bf16(out, (rows, d))
    assert np.all(np.abs(got - want) <= 2.0 ** -7 * np.abs(want) + 1e-6)
    assert np.all(np.abs(lse.host(np.float32, (rows,)) - (pl.max(axis=0) + np.log(w.sum(0)))) <= 1e-4)


@pytest.mark.parametrize("nbytes", [16, 4096 + 16, 1 << 20])
def test_ring_step_stays_inside(lib, bands, nbytes):
    import torch
    n = nbytes // 4
    rng = np.random.default_rng(nbytes)
    own, recv = rng.standard_normal(n).astype(np.float32), rng.standard_normal(n).astype(np.float32)
    down, drecv = Banded.of(own), Banded.of(recv)
    dst = Banded(nbytes, fill=0xC0)
    flag, status = Banded.of(np.ones(1, np.uint32)), Banded.of(np.zeros(1, np.uint32))
    st = torch.cuda.current_stream().cuda_stream
    lib.libra_ring_step(0, dst.ptr, down.ptr, drecv.ptr, nbytes, lib.RING_F32, flag.ptr, 1, 100000, status.ptr, 2, st)
    all_intact(bands)
    assert status.host(np.uint32, (1,))[0] == 0
    assert np.array_equal(dst.host(np.float32, (n,)), own + recv)
    lib.libra_ring_step(0, down.ptr, down.ptr, drecv.ptr, nbytes, lib.RING_F32, flag.ptr, 1, 100000, status.ptr, 2, st)   # in place
    all_intact(bands)
    assert np.array_equal(down.host(np.float32, (n,)), own + recv)
