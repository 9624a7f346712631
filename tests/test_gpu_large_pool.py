"""Pools whose element and byte offsets pass 2^31 and 2^32: the step, the fused append and the KV move copies
on pages at the top of a 5 GB pool give the same bits as on a compact pool (page placement never changes a
result), match the oracle, and write nothing outside the pages they own."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from oracle import kv_move_oracle as M
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu

HQ, HKV, D = 32, 8, 128
NUM_PAGES = 160_000           # x 8 heads x 16 tokens x 128 = 2.62e9 elements, 5.24e9 bytes per bf16 pool
NUM_PAGES_8BIT = 300_000      # the same memory seen as an 8-bit pool: 4.9e9 bytes
LENS = [2500, 17, 1, 700, 0, 4097]


def top_pages(n, num_pages, seed):
    """n distinct page ids, most from the last tenth of the pool, a few from its start."""
    rng = np.random.default_rng(seed)
    hi = rng.choice(np.arange(num_pages - num_pages // 10, num_pages), size=n, replace=False)
    hi[:: 7] = rng.choice(np.arange(0, 1000), size=len(hi[:: 7]), replace=False)
    return hi.astype(np.int64)


def remap(bt, ids):
    return np.where(bt >= 0, ids[np.maximum(bt, 0)], -1).astype(np.int32)


def changed_pages(a, b):
    """Ids of the pages in which two device pools differ."""
    import torch
    diff = (a != b).flatten(1).any(dim=1)
    return set(torch.nonzero(diff).flatten().cpu().tolist())


def test_offsets_beyond_32_bits_bf16(lib):
    import torch
    dev = torch.device("cuda:0")
    B = len(LENS)
    lens_a, bt, q, k, v = W.random_case(301, B, HQ, HKV, D, LENS)
    small = H.run_host_case(lib, q, k, v, bt, lens_a)
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens_a)

    ids = top_pages(k.shape[0], NUM_PAGES, 1)
    assert int(ids.max()) * HKV * 16 * D > 2 ** 31
    bt_big = remap(bt, ids)
    idx = torch.from_numpy(ids).to(dev)
    kbig = torch.zeros((NUM_PAGES, HKV, 16, D), dtype=torch.int16, device=dev)
    vbig = torch.zeros((NUM_PAGES, HKV, 16, D), dtype=torch.int16, device=dev)
    kbig[idx] = H.to_dev(k, dev)
    vbig[idx] = H.to_dev(v, dev)

    r = H.Runner(lib, HQ, HKV, D, NUM_PAGES, B, bt.shape[1])
    dq, dbt = H.to_dev(q, dev), H.to_dev(bt_big, dev)
    got = H.bf16_dev_to_f32(r.run(dq, kbig, vbig, dbt, lens_a))
    assert np.array_equal(got, small)
    assert gates.stated_violations(got, ref) == 0 and gates.tight_violations(got, ref) == 0

    # fused append: the newest token's rows land in the right page of the large pool and nowhere else
    rng = np.random.default_rng(6)
    k_new = W.f32_to_bf16_bits(rng.standard_normal((B, HKV, D), dtype=np.float32))
    v_new = W.f32_to_bf16_bits(rng.standard_normal((B, HKV, D), dtype=np.float32))
    k_ref, v_ref = k.copy(), v.copy()
    last_pages = set()
    for b, L in enumerate(LENS):
        if L:
            k_ref[bt[b, (L - 1) // 16], :, (L - 1) % 16, :] = k_new[b]
            v_ref[bt[b, (L - 1) // 16], :, (L - 1) % 16, :] = v_new[b]
            last_pages.add(int(bt_big[b, (L - 1) // 16]))
    ref2, _ = O.paged_decode_attention(q, k_ref, v_ref, bt, lens_a)
    k_before, v_before = kbig.clone(), vbig.clone()
    dl = torch.from_numpy(lens_a.copy()).to(dev)
    out = torch.full((B, HQ, D), H.CANARY, dtype=torch.int16, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    r.h.plan(lens_a, r.ws.data_ptr(), r.ws.numel(), st)
    dkn, dvn = H.to_dev(k_new, dev), H.to_dev(v_new, dev)    # kept alive until the kernel has run
    r.h.decode_attn_append(dq.data_ptr(), dkn.data_ptr(), dvn.data_ptr(),
                           kbig.data_ptr(), vbig.data_ptr(), dbt.data_ptr(), dl.data_ptr(), out.data_ptr(), st)
    torch.cuda.synchronize()
    assert r.h.debug_error_word() == 0
    got2 = H.bf16_dev_to_f32(out)
    assert gates.stated_violations(got2, ref2) == 0 and gates.tight_violations(got2, ref2) == 0
    assert np.array_equal(kbig[idx].cpu().numpy().view(np.uint16), k_ref)
    assert np.array_equal(vbig[idx].cpu().numpy().view(np.uint16), v_ref)
    assert changed_pages(kbig, k_before) <= last_pages and changed_pages(vbig, v_before) <= last_pages
    del k_before, v_before

    # KV move: gather from the top of the pool, scatter to other pages there under a new placement
    offs = np.concatenate([[0], np.cumsum(lens_a.astype(np.int64))])
    total = int(offs[-1])
    doffs = torch.from_numpy(offs[:-1].copy()).to(dev)
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    h0, hn = 2, 4
    k_dense = torch.full((total, hn, D), 0x7FC0, dtype=torch.int16, device=dev)
    v_dense = torch.full((total, hn, D), 0x7FC0, dtype=torch.int16, device=dev)
    r.h.kv_gather(kbig.data_ptr(), vbig.data_ptr(), dbt.data_ptr(), dl.data_ptr(), doffs.data_ptr(), B, max(LENS),
                  h0, hn, k_dense.data_ptr(), v_dense.data_ptr(), err.data_ptr(), st)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    assert np.array_equal(k_dense.cpu().numpy().view(np.uint16), M.gather(k_ref, bt, lens_a, h0, hn))
    assert np.array_equal(v_dense.cpu().numpy().view(np.uint16), M.gather(v_ref, bt, lens_a, h0, hn))

    free = np.setdiff1d(np.arange(NUM_PAGES - 12000, NUM_PAGES), ids)
    ids2 = np.random.default_rng(2).choice(free, size=k.shape[0], replace=False).astype(np.int64)
    bt2 = remap(bt, ids2)
    k_before, v_before = kbig.clone(), vbig.clone()
    dbt2 = H.to_dev(bt2, dev)
    r.h.kv_scatter(k_dense.data_ptr(), v_dense.data_ptr(), dbt2.data_ptr(), dl.data_ptr(),
                   doffs.data_ptr(), B, max(LENS), h0, hn, kbig.data_ptr(), vbig.data_ptr(), err.data_ptr(), st)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    want_k = np.zeros_like(k)
    want_v = np.zeros_like(v)
    M.scatter(M.gather(k_ref, bt, lens_a, h0, hn), want_k, bt, lens_a, h0)   # small pool, old ids = rows of ids2
    M.scatter(M.gather(v_ref, bt, lens_a, h0, hn), want_v, bt, lens_a, h0)
    idx2 = torch.from_numpy(ids2).to(dev)
    assert np.array_equal(kbig[idx2].cpu().numpy().view(np.uint16), want_k)
    assert np.array_equal(vbig[idx2].cpu().numpy().view(np.uint16), want_v)
    owned = {int(x) for x in bt2[bt2 >= 0]}
    assert changed_pages(kbig, k_before) <= owned and changed_pages(vbig, v_before) <= owned
    r.h.close()


def test_offsets_beyond_32_bits_8bit_cache(lib):
    import torch
    dev = torch.device("cuda:0")
    B = len(LENS)
    lens_a, bt, q, k8, v8 = W.random_case_e4m3(302, B, HQ, HKV, D, LENS)
    ref, _ = O.paged_decode_attention_fp8(q, k8, v8, bt, lens_a, 0.5, 2.0)
    ids = top_pages(k8.shape[0], NUM_PAGES_8BIT, 3)
    assert int(ids.max()) * HKV * 16 * D > 2 ** 32
    bt_big = remap(bt, ids)
    idx = torch.from_numpy(ids).to(dev)
    kbig = torch.zeros((NUM_PAGES_8BIT, HKV, 16, D), dtype=torch.uint8, device=dev)
    vbig = torch.zeros((NUM_PAGES_8BIT, HKV, 16, D), dtype=torch.uint8, device=dev)
    kbig[idx] = torch.from_numpy(k8).to(dev)
    vbig[idx] = torch.from_numpy(v8).to(dev)

    outs = []
    for pool_k, pool_v, table, pages in ((torch.from_numpy(k8).to(dev), torch.from_numpy(v8).to(dev), bt, k8.shape[0]),
                                         (kbig, vbig, bt_big, NUM_PAGES_8BIT)):
        h = lib.Handle(HQ, HKV, D, pages, B, bt.shape[1])
        h.set_kv_dtype(lib.KV_E4M3, 0.5, 2.0)
        ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
        dq, dbt = H.to_dev(q, dev), H.to_dev(table, dev)
        dl = torch.from_numpy(lens_a.copy()).to(dev)
        out = torch.full((B, HQ, D), H.CANARY, dtype=torch.int16, device=dev)
        st = torch.cuda.current_stream().cuda_stream
        h.plan(lens_a, ws.data_ptr(), ws.numel(), st)
        h.decode_attn(dq.data_ptr(), pool_k.data_ptr(), pool_v.data_ptr(), dbt.data_ptr(), dl.data_ptr(),
                      out.data_ptr(), st)
        torch.cuda.synchronize()
        assert h.debug_error_word() == 0
        outs.append(H.bf16_dev_to_f32(out))
        h.close()
    assert np.array_equal(outs[0], outs[1])
    assert gates.stated_violations(outs[1], ref) == 0 and gates.tight_violations(outs[1], ref) == 0


def test_largest_batch(lib):
    """The largest batch a handle takes (2^18 sequences, the width of the plan's sequence field): short ragged
    sequences incl. empty ones, a plan far too large for the kernel parameters, half a million thread blocks;
    sampled rows against the oracle, every row written, empty rows zero."""
    import torch
    dev = torch.device("cuda:0")
    B, Hq, Hkv, d = 1 << 18, 4, 2, 64
    rng = np.random.default_rng(77)
    lens = rng.integers(0, 33, size=B).astype(np.int32)          # 0 .. 32 tokens: one or two pages
    lens[:5] = [0, 1, 16, 17, 32]
    n_pages = (lens.astype(np.int64) + 15) // 16
    first = np.concatenate([[0], np.cumsum(n_pages)[:-1]])
    total_pages = int(n_pages.sum())
    perm = rng.permutation(total_pages).astype(np.int32)
    bt = np.full((B, 2), -1, dtype=np.int32)
    for j in range(2):
        has = n_pages > j
        bt[has, j] = perm[first[has] + j]
    gen = torch.Generator(device=dev).manual_seed(5)
    k = torch.randn((total_pages, Hkv, 16, d), device=dev, generator=gen).to(torch.bfloat16)
    v = torch.randn((total_pages, Hkv, 16, d), device=dev, generator=gen).to(torch.bfloat16)
    q = torch.randn((B, Hq, d), device=dev, generator=gen).to(torch.bfloat16)
    with pytest.raises(lib.LibraError):
        lib.Handle(Hq, Hkv, d, total_pages, B + 1, 2)             # one more than the plan format holds
    r = H.Runner(lib, Hq, Hkv, d, total_pages, B, 2)
    out = H.bf16_dev_to_f32(r.run(q, k, v, H.to_dev(bt, dev), lens))
    assert np.all(np.isfinite(out))                               # every row written (the canary is a NaN)
    assert np.all(out[lens == 0] == 0.0)
    assert len(r.h.plan_export()["items"]) == int((lens > 0).sum())
    rows = [0, 1, 2, 3, 4, B - 1] + [int(x) for x in rng.choice(B, size=300, replace=False)]
    kh, vh, bth, lh = H.gather_for_oracle(k, v, bt, lens, rows)
    qh = q.view(torch.int16)[torch.tensor(rows, device=dev)].cpu().numpy().view(np.uint16)
    ref, _ = O.paged_decode_attention(qh, kh, vh, bth, lh)
    got = out[rows]
    assert gates.stated_violations(got, ref) == 0 and gates.tight_violations(got, ref) == 0
    r.h.close()
