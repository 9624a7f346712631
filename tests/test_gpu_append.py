"""The decode step with the KV append fused in (libra_decode_attn_append) against the definition: write
the new token's K and V rows into slot (L-1) % 16 of the sequence's last page, then attend.  The
attention output is compared with the float64 oracle on the updated pools, and the pools the kernel
leaves behind must equal the updated pools bit for bit."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu


def reference_append(k, v, bt, lens, k_new, v_new):
    k2, v2 = k.copy(), v.copy()
    P = k.shape[2]
    for b, L in enumerate(lens):
        L = int(L)
        if L == 0:
            continue
        page, slot = bt[b, (L - 1) // P], (L - 1) % P
        k2[page, :, slot, :] = k_new[b]
        v2[page, :, slot, :] = v_new[b]
    return k2, v2


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("Hq,Hkv,d,lens,P", [
    (8, 2, 128, [1, 16, 17, 32, 33, 700], 16),
    (32, 8, 128, [5000, 1300, 0, 2049], 16),
    (4, 1, 64, [300, 64, 7, 1], 16),
    (40, 8, 128, [48, 1025], 16),
    (8, 2, 128, [1, 17, 32, 33, 64, 65, 700], 64),
    (8, 2, 128, [31, 32, 33, 1000], 32),
])
def test_append_matches_definition(lib, Hq, Hkv, d, lens, P, layout):
    import torch
    dev = torch.device("cuda:0")
    B = len(lens)
    lens_a, bt, q, k, v = W.random_case(77, B, Hq, Hkv, d, lens, page_size=P)   # the new token's slot holds poison
    for b, L in enumerate(lens):                                   # make sure of it even though the slot is "owned"
        if L:
            k[bt[b, (L - 1) // P], :, (L - 1) % P, :] = W.f32_to_bf16_bits(np.array([W.POISON_F32]))[0]
            v[bt[b, (L - 1) // P], :, (L - 1) % P, :] = W.f32_to_bf16_bits(np.array([-W.POISON_F32]))[0]
    rng = np.random.default_rng(5)
    k_new = W.f32_to_bf16_bits(rng.standard_normal((B, Hkv, d), dtype=np.float32))
    v_new = W.f32_to_bf16_bits(rng.standard_normal((B, Hkv, d), dtype=np.float32))
    k_ref, v_ref = reference_append(k, v, bt, lens_a, k_new, v_new)
    ref, _ = O.paged_decode_attention(q, k_ref, v_ref, bt, lens_a)

    for plan in (None, lib.PlanParams(4, 1, 2, 64, 64, 64)):
        kd = k if layout == "HND" else np.ascontiguousarray(k.transpose(0, 2, 1, 3))
        vd = v if layout == "HND" else np.ascontiguousarray(v.transpose(0, 2, 1, 3))
        r = H.Runner(lib, Hq, Hkv, d, k.shape[0], B, bt.shape[1], layout, plan, page_size=P)
        dq, dk, dv, dbt, dkn, dvn = (H.to_dev(x, dev) for x in (q, kd, vd, bt, k_new, v_new))
        dl = torch.from_numpy(lens_a.copy()).to(dev)
        out = torch.full((B, Hq, d), H.CANARY, dtype=torch.int16, device=dev)
        st = torch.cuda.current_stream().cuda_stream
        r.h.plan(lens_a, r.ws.data_ptr(), r.ws.numel(), st)
        r.h.decode_attn_append(dq.data_ptr(), dkn.data_ptr(), dvn.data_ptr(), dk.data_ptr(), dv.data_ptr(),
                               dbt.data_ptr(), dl.data_ptr(), out.data_ptr(), st)
        torch.cuda.synchronize()
        assert r.h.debug_error_word() == 0
        got = H.bf16_dev_to_f32(out)
        assert np.all(np.isfinite(got))
        assert gates.stated_violations(got, ref) == 0
        assert gates.tight_violations(got, ref) == 0, gates.tight_ratio(got, ref)
        k_after = dk.cpu().numpy().view(np.uint16)
        v_after = dv.cpu().numpy().view(np.uint16)
        if layout == "NHD":
            k_after, v_after = k_after.transpose(0, 2, 1, 3), v_after.transpose(0, 2, 1, 3)
        assert np.array_equal(k_after, k_ref) and np.array_equal(v_after, v_ref)
        r.h.close()


def test_chain_of_append_steps_with_early_prefetch(lib):
    """Five decode steps with the fused append, lengths growing by one per step, queued without synchronising:
    with early prefetch the step may start its copies while the previous step (which wrote the previous token's
    rows) is still running; outputs and pools must equal the default's bit for bit, and the oracle's."""
    import torch
    dev = torch.device("cuda:0")
    steps = 5
    lens0 = np.array([1, 15, 16, 31, 300, 1024, 2047], dtype=np.int32)
    B, Hq, Hkv, d = len(lens0), 16, 4, 128
    lens_max, bt, q, k, v = W.random_case(81, B, Hq, Hkv, d, lens0 + steps, poison=False)
    rng = np.random.default_rng(82)
    new_k = W.f32_to_bf16_bits(rng.standard_normal((steps, B, Hkv, d)).astype(np.float32))
    new_v = W.f32_to_bf16_bits(rng.standard_normal((steps, B, Hkv, d)).astype(np.float32))
    new_q = W.f32_to_bf16_bits(rng.standard_normal((steps, B, Hq, d)).astype(np.float32))
    res = {}
    for early in (False, True):
        r = H.Runner(lib, Hq, Hkv, d, k.shape[0], B, bt.shape[1], plan=lib.PlanParams(148, 1, 1, 256, 512, 64))
        r.h.set_early_prefetch(early)
        kd, vd, btd = H.to_dev(k, dev), H.to_dev(v, dev), H.to_dev(bt, dev)
        nk, nv, nq = H.to_dev(new_k, dev), H.to_dev(new_v, dev), H.to_dev(new_q, dev)
        lens_dev = [torch.from_numpy(lens0 + 1 + i).to(dev) for i in range(steps)]
        outs = torch.zeros((steps, B, Hq, d), dtype=torch.int16, device=dev)
        st = torch.cuda.current_stream().cuda_stream
        torch.cuda.synchronize()
        for i in range(steps):
            r.h.plan(lens0 + 1 + i, r.ws.data_ptr(), r.ws.numel(), st)
            r.h.decode_attn_append(nq[i].data_ptr(), nk[i].data_ptr(), nv[i].data_ptr(), kd.data_ptr(), vd.data_ptr(),
                                   btd.data_ptr(), lens_dev[i].data_ptr(), outs[i].data_ptr(), st)
        torch.cuda.synchronize()
        assert r.h.debug_error_word() == 0
        res[early] = (H.bf16_dev_to_f32(outs), kd.cpu().numpy().view(np.uint16), vd.cpu().numpy().view(np.uint16))
        r.h.close()
    assert np.array_equal(res[True][0], res[False][0])
    assert np.array_equal(res[True][1], res[False][1]) and np.array_equal(res[True][2], res[False][2])
    kk, vv = k.copy(), v.copy()
    for i in range(steps):
        for b in range(B):
            t = int(lens0[b]) + i
            kk[bt[b, t // 16], :, t % 16] = new_k[i, b]
            vv[bt[b, t // 16], :, t % 16] = new_v[i, b]
    assert np.array_equal(res[True][1], kk) and np.array_equal(res[True][2], vv)
    ref, _ = O.paged_decode_attention(new_q[-1], kk, vv, bt, lens0 + steps)
    got = res[True][0][-1]
    assert gates.stated_violations(got, ref) == 0 and gates.tight_violations(got, ref) == 0
