"""KV gather / scatter on the GPU against the explicit-index oracle (byte-exact), for both pool layouts,
and the end-to-end property the paper's migration relies on: after resharding a request's KV along the
head dimension (TP 1 -> 2 and back), decode attention on the shards gives the same bits as before."""
import numpy as np
import pytest

from oracle import kv_move_oracle as M
from paper_2606_03077_b200 import workloads as W

import gpu_harness as H

pytestmark = pytest.mark.gpu


def dev_i64(a, dev):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int64)).to(dev)


@pytest.mark.parametrize("layout", ["HND", "NHD"])
@pytest.mark.parametrize("Hkv,d,lens,h0,hn,P", [
    (8, 128, [1, 16, 17, 700, 0, 2049], 0, 8, 16),
    (8, 128, [333, 64], 2, 4, 16),
    (4, 64, [40, 5, 1000], 3, 1, 16),
    (4, 128, [1, 33, 64, 65, 700], 1, 2, 64),
])
def test_gather_and_scatter_are_exact(lib, Hkv, d, lens, h0, hn, P, layout):
    import torch
    dev = torch.device("cuda:0")
    B = len(lens)
    lens_a, bt, q, k, v = W.random_case(91, B, Hkv, Hkv, d, lens, poison=False, page_size=P)
    kd = k if layout == "HND" else np.ascontiguousarray(k.transpose(0, 2, 1, 3))
    vd = v if layout == "HND" else np.ascontiguousarray(v.transpose(0, 2, 1, 3))
    strides = (0, 0, 0) if layout == "HND" else (P * Hkv * d, d, Hkv * d)
    h = lib.Handle(Hkv, Hkv, d, k.shape[0], B, bt.shape[1], page_size=P, kv_strides=strides)
    offs = np.concatenate([[0], np.cumsum(lens_a.astype(np.int64))])
    total = int(offs[-1])
    dk, dv, dbt = (H.to_dev(x, dev) for x in (kd, vd, bt))
    dl = torch.from_numpy(lens_a.copy()).to(dev)
    doffs = dev_i64(offs[:-1], dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    k_dense = torch.full((total, hn, d), 0x7FC0, dtype=torch.int16, device=dev)
    v_dense = torch.full((total, hn, d), 0x7FC0, dtype=torch.int16, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    h.kv_gather(dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(), doffs.data_ptr(), B, int(lens_a.max()),
                h0, hn, k_dense.data_ptr(), v_dense.data_ptr(), err.data_ptr(), st)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    assert np.array_equal(k_dense.cpu().numpy().view(np.uint16), M.gather(k, bt, lens_a, h0, hn))
    assert np.array_equal(v_dense.cpu().numpy().view(np.uint16), M.gather(v, bt, lens_a, h0, hn))

    # scatter the shard into a fresh pool under a new placement, at head offset 0 of a pool with hn heads
    rng = np.random.default_rng(4)
    bt2, pool2 = W.draw_block_table(lens_a, int(W.pages_needed(lens_a, P).sum()) + 5, rng, page_size=P, ld=bt.shape[1])
    strides2 = (0, 0, 0) if layout == "HND" else (P * hn * d, d, hn * d)
    h2 = lib.Handle(hn, hn, d, pool2, B, bt.shape[1], page_size=P, kv_strides=strides2)
    shape2 = (pool2, hn, P, d) if layout == "HND" else (pool2, P, hn, d)
    k2 = torch.full(shape2, -1, dtype=torch.int16, device=dev)
    v2 = torch.full(shape2, -1, dtype=torch.int16, device=dev)
    dbt2 = H.to_dev(bt2, dev)
    h2.kv_scatter(k_dense.data_ptr(), v_dense.data_ptr(), dbt2.data_ptr(), dl.data_ptr(), doffs.data_ptr(),
                  B, int(lens_a.max()), 0, hn, k2.data_ptr(), v2.data_ptr(), err.data_ptr(), st)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    want_k = np.full((pool2, hn, P, d), 0xFFFF, np.uint16)
    want_v = np.full((pool2, hn, P, d), 0xFFFF, np.uint16)
    M.scatter(M.gather(k, bt, lens_a, h0, hn), want_k, bt2, lens_a, 0)
    M.scatter(M.gather(v, bt, lens_a, h0, hn), want_v, bt2, lens_a, 0)
    got_k = k2.cpu().numpy().view(np.uint16)
    got_v = v2.cpu().numpy().view(np.uint16)
    if layout == "NHD":
        got_k, got_v = got_k.transpose(0, 2, 1, 3), got_v.transpose(0, 2, 1, 3)
    assert np.array_equal(got_k, want_k) and np.array_equal(got_v, want_v)   # untouched slots still 0xFFFF
    h.close(); h2.close()


def test_bad_page_id_is_skipped_and_flagged(lib):
    import torch
    dev = torch.device("cuda:0")
    lens_a, bt, q, k, v = W.random_case(92, 1, 2, 2, 128, [40], poison=False)
    bad = bt.copy(); bad[0, 1] = k.shape[0] + 3
    h = lib.Handle(2, 2, 128, k.shape[0], 1, bt.shape[1])
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    kd = torch.zeros((40, 2, 128), dtype=torch.int16, device=dev); vd = torch.zeros_like(kd)
    dk, dv, dbad = (H.to_dev(x, dev) for x in (k, v, bad))    # kept alive until the kernel has run
    dl = torch.tensor([40], dtype=torch.int32, device=dev)
    doffs = dev_i64([0], dev)
    h.kv_gather(dk.data_ptr(), dv.data_ptr(), dbad.data_ptr(), dl.data_ptr(), doffs.data_ptr(), 1, 40, 0, 2,
                kd.data_ptr(), vd.data_ptr(), err.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert int(err.item()) & lib.ERR_BAD_PAGE_ID
    assert np.array_equal(kd.cpu().numpy().view(np.uint16)[:16], M.gather(k, bt, [16], 0, 2))
    h.close()


def test_decode_is_unchanged_by_a_head_reshard(lib):
    """TP 1 -> 2: the pool's 8 KV heads become two 4-head pools on new pages; decode on each shard with its
    16 query heads returns the bits the unsharded decode returned for those heads.  Then TP 2 -> 1."""
    import torch
    dev = torch.device("cuda:0")
    lens = [3000, 17, 1025, 1]
    Hq, Hkv, d, B = 32, 8, 128, 4
    lens_a, bt, q, k, v = W.random_case(93, B, Hq, Hkv, d, lens)
    prm = lib.PlanParams(148, 2, 4, 256, 256, 64)   # fixed constants: same chunking whatever the head count
    base = H.run_host_case(lib, q, k, v, bt, lens_a, plan=prm)

    offs = np.concatenate([[0], np.cumsum(lens_a.astype(np.int64))])
    total = int(offs[-1])
    st = torch.cuda.current_stream().cuda_stream
    src = lib.Handle(Hq, Hkv, d, k.shape[0], B, bt.shape[1])
    dk, dv, dbt = (H.to_dev(x, dev) for x in (k, v, bt))
    dl = torch.from_numpy(lens_a.copy()).to(dev)
    doffs = dev_i64(offs[:-1], dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    rng = np.random.default_rng(8)
    back_k = torch.zeros((k.shape[0], Hkv, 16, d), dtype=torch.int16, device=dev)
    back_v = torch.zeros_like(back_k)
    for r in range(2):
        kd = torch.empty((total, 4, d), dtype=torch.int16, device=dev); vd = torch.empty_like(kd)
        src.kv_gather(dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(), doffs.data_ptr(), B, max(lens),
                      4 * r, 4, kd.data_ptr(), vd.data_ptr(), err.data_ptr(), st)
        bt2, pool2 = W.draw_block_table(lens_a, int(W.pages_needed(lens_a).sum()) + 9, rng, ld=bt.shape[1])
        tgt = lib.Handle(Hq // 2, 4, d, pool2, B, bt.shape[1], plan=prm)
        k2 = torch.full((pool2, 4, 16, d), 0x7F80, dtype=torch.int16, device=dev)   # +inf everywhere a slot is not written
        v2 = torch.full_like(k2, 0x7F80)
        dbt2 = H.to_dev(bt2, dev)
        tgt.kv_scatter(kd.data_ptr(), vd.data_ptr(), dbt2.data_ptr(), dl.data_ptr(), doffs.data_ptr(), B, max(lens), 0, 4,
                       k2.data_ptr(), v2.data_ptr(), err.data_ptr(), st)
        ws = torch.empty(tgt.workspace_size(), dtype=torch.uint8, device=dev)
        out = torch.full((B, Hq // 2, d), H.CANARY, dtype=torch.int16, device=dev)
        q_r = H.to_dev(np.ascontiguousarray(q[:, 16 * r:16 * r + 16]), dev)
        tgt.plan(lens_a, ws.data_ptr(), ws.numel(), st)
        tgt.decode_attn(q_r.data_ptr(), k2.data_ptr(), v2.data_ptr(), dbt2.data_ptr(), dl.data_ptr(), out.data_ptr(), st)
        torch.cuda.synchronize()
        assert tgt.debug_error_word() == 0 and int(err.item()) == 0
        assert np.array_equal(H.bf16_dev_to_f32(out), base[:, 16 * r:16 * r + 16])
        # TP 2 -> 1: concatenate the shard back into an 8-head pool at head offset 4 r
        kd2 = torch.empty_like(kd); vd2 = torch.empty_like(vd)
        tgt.kv_gather(k2.data_ptr(), v2.data_ptr(), dbt2.data_ptr(), dl.data_ptr(), doffs.data_ptr(), B, max(lens), 0, 4,
                      kd2.data_ptr(), vd2.data_ptr(), err.data_ptr(), st)
        src.kv_scatter(kd2.data_ptr(), vd2.data_ptr(), dbt.data_ptr(), dl.data_ptr(), doffs.data_ptr(), B, max(lens),
                       4 * r, 4, back_k.data_ptr(), back_v.data_ptr(), err.data_ptr(), st)
        torch.cuda.synchronize()
        tgt.close()
    r8 = H.Runner(lib, Hq, Hkv, d, k.shape[0], B, bt.shape[1], plan=prm)
    again = H.bf16_dev_to_f32(r8.run(H.to_dev(q, dev), back_k, back_v, dbt, lens_a))
    assert np.array_equal(again, base)
    r8.h.close(); src.close()


def test_offload_to_pinned_host_memory_and_reload(lib):
    """The dense buffer in pinned host memory (the paper's offload target): the gather kernel writes it over the bus,
    the scatter kernel reads it back into a pool with a new page placement; both exact."""
    import torch
    dev = torch.device("cuda:0")
    lens = [700, 33, 1, 2049]
    B, Hkv, d = len(lens), 4, 128
    lens_a, bt, q, k, v = W.random_case(95, B, Hkv, Hkv, d, lens, poison=False)
    h = lib.Handle(Hkv, Hkv, d, k.shape[0], B, bt.shape[1])
    offs = np.concatenate([[0], np.cumsum(lens_a.astype(np.int64))])
    total = int(offs[-1])
    dk, dv, dbt = (H.to_dev(x, dev) for x in (k, v, bt))
    dl = torch.from_numpy(lens_a.copy()).to(dev)
    doffs = dev_i64(offs[:-1], dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    k_host = torch.full((total, Hkv, d), 0x7FC0, dtype=torch.int16).pin_memory()
    v_host = torch.full((total, Hkv, d), 0x7FC0, dtype=torch.int16).pin_memory()
    st = torch.cuda.current_stream().cuda_stream
    h.kv_gather(dk.data_ptr(), dv.data_ptr(), dbt.data_ptr(), dl.data_ptr(), doffs.data_ptr(), B, int(lens_a.max()),
                0, Hkv, k_host.data_ptr(), v_host.data_ptr(), err.data_ptr(), st)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    assert np.array_equal(k_host.numpy().view(np.uint16), M.gather(k, bt, lens_a, 0, Hkv))
    assert np.array_equal(v_host.numpy().view(np.uint16), M.gather(v, bt, lens_a, 0, Hkv))
    rng = np.random.default_rng(6)
    bt2, pool2 = W.draw_block_table(lens_a, int(W.pages_needed(lens_a).sum()) + 3, rng, ld=bt.shape[1])
    h2 = lib.Handle(Hkv, Hkv, d, pool2, B, bt.shape[1])
    k2 = torch.full((pool2, Hkv, 16, d), -1, dtype=torch.int16, device=dev)
    v2 = torch.full((pool2, Hkv, 16, d), -1, dtype=torch.int16, device=dev)
    dbt2 = H.to_dev(bt2, dev)
    h2.kv_scatter(k_host.data_ptr(), v_host.data_ptr(), dbt2.data_ptr(), dl.data_ptr(), doffs.data_ptr(), B,
                  int(lens_a.max()), 0, Hkv, k2.data_ptr(), v2.data_ptr(), err.data_ptr(), st)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    want_k = np.full((pool2, Hkv, 16, d), 0xFFFF, np.uint16)
    want_v = np.full((pool2, Hkv, 16, d), 0xFFFF, np.uint16)
    M.scatter(M.gather(k, bt, lens_a, 0, Hkv), want_k, bt2, lens_a, 0)
    M.scatter(M.gather(v, bt, lens_a, 0, Hkv), want_v, bt2, lens_a, 0)
    assert np.array_equal(k2.cpu().numpy().view(np.uint16), want_k)
    assert np.array_equal(v2.cpu().numpy().view(np.uint16), want_v)
    h.close(); h2.close()
