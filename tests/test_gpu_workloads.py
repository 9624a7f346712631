"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times: the four
large workloads with pools filled on the device, compared with the oracle element by element on EVERY
sequence of every step (the used pages are copied back group by group; the float64 oracle needs seconds
per workload).  The E4M3 cache and the several-query-token step are checked the same way."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu


WORST = {}   # (test, workload, step) -> (max abs err, worst tight-gate ratio), printed at the end of the module


@pytest.fixture(scope="module", autouse=True)
def report_worst():
    yield
    for key, (a, r) in sorted(WORST.items()):
        print(f"\nfull-size parity {key}: max abs err {a:.3e}, worst tight-gate ratio {r:.3f}")


@pytest.mark.parametrize("name", ["lognormal_b64", "longtail_mix_b256", "straggler_b8", "shift_b128"])
def test_workload_parity(lib, name):
    import torch
    dev = torch.device("cuda:0")
    w = W.WORKLOADS[name]
    lay0, _ = W.make_layout(name, 0)
    q, k, v = W.fill_device_pools(lay0, dev, poison=False)
    ld = max(W.make_layout(name, s)[0].block_table.shape[1] for s in range(w.steps))
    r = H.Runner(lib, w.num_q_heads, w.num_kv_heads, w.head_dim, lay0.pool_pages, w.batch, ld)
    for step in range(w.steps):
        lay, _ = W.make_layout(name, step)
        saved = W.poison_tails(lay, k, v)  # new lengths and page placement over the same pool contents
        bt = np.full((w.batch, ld), -1, dtype=np.int32)
        bt[:, :lay.block_table.shape[1]] = lay.block_table
        out = H.bf16_dev_to_f32(r.run(q, k, v, H.to_dev(bt, dev), lay.seq_lens))
        assert np.all(np.isfinite(out))
        WORST[("bf16", name, step)] = H.compare_every_sequence(
            out, q, k, v, bt, lay.seq_lens, lambda *a: O.paged_decode_attention(*a)[0], gates)
        for mode in (0, 1):           # step C as its own kernel / inside the decode kernel: same bits
            r.h.set_combine_mode(mode)
            out2 = H.bf16_dev_to_f32(r.run(q, k, v, H.to_dev(bt, dev), lay.seq_lens))
            assert np.array_equal(out, out2)
        r.h.set_combine_mode(1)
        W.restore_tails(saved, k, v)
    r.h.close()


@pytest.mark.parametrize("name", ["lognormal_b64", "longtail_mix_b256", "straggler_b8"])
def test_workload_parity_8bit_cache(lib, name):
    """The same full-size workloads over an E4M3 cache (device pools of random finite codes, default launch
    configuration), every sequence against the oracle."""
    import torch
    dev = torch.device("cuda:0")
    w = W.WORKLOADS[name]
    lay, _ = W.make_layout(name, 0)
    shape = (lay.pool_pages, w.num_kv_heads, w.page_size, w.head_dim)
    gen = torch.Generator(device=dev).manual_seed(11)

    def codes():   # sign and mantissa random, exponent field 0..8: finite, |x| < 4
        r = torch.randint(0, 256, shape, dtype=torch.uint8, device=dev, generator=gen)
        r &= 0x87
        r |= torch.randint(0, 9, shape, dtype=torch.uint8, device=dev, generator=gen) << 3
        return r

    k8, v8 = codes(), codes()
    q = torch.randn((w.batch, w.num_q_heads, w.head_dim), device=dev, generator=gen).to(torch.bfloat16)
    h = lib.Handle(w.num_q_heads, w.num_kv_heads, w.head_dim, lay.pool_pages, w.batch, lay.block_table.shape[1])
    h.set_kv_dtype(lib.KV_E4M3, 0.5, 1.25)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
    btd = H.to_dev(lay.block_table, dev)
    lens_dev = torch.from_numpy(lay.seq_lens.copy()).to(dev)
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), H.CANARY, dtype=torch.int16, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    h.plan(lay.seq_lens, ws.data_ptr(), ws.numel(), st)
    h.decode_attn(q.data_ptr(), k8.data_ptr(), v8.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(), out.data_ptr(), st)
    torch.cuda.synchronize()
    assert h.debug_error_word() == 0
    got_all = H.bf16_dev_to_f32(out)
    assert np.all(np.isfinite(got_all))
    WORST[("e4m3", name, 0)] = H.compare_every_sequence(
        got_all, q, k8, v8, lay.block_table, lay.seq_lens,
        lambda *a: O.paged_decode_attention_fp8(*a, 0.5, 1.25)[0], gates)
    h.close()


@pytest.mark.parametrize("name,q_len", [("lognormal_b64", 4), ("straggler_b8", 2), ("shift_b128", 3)])
def test_workload_parity_several_query_tokens(lib, name, q_len):
    """The full-size workloads with q_len query tokens per sequence, every sequence against the oracle."""
    import torch
    dev = torch.device("cuda:0")
    w = W.WORKLOADS[name]
    lay, _ = W.make_layout(name, 0)
    _, k, v = W.fill_device_pools(lay, dev, poison=True)
    gen = torch.Generator(device=dev).manual_seed(12)
    q = torch.randn((w.batch, q_len, w.num_q_heads, w.head_dim), device=dev, generator=gen).to(torch.bfloat16)
    h = lib.Handle(w.num_q_heads, w.num_kv_heads, w.head_dim, lay.pool_pages, w.batch, lay.block_table.shape[1])
    h.set_max_query_tokens(q_len)
    ws = torch.empty(h.workspace_size(), dtype=torch.uint8, device=dev)
    btd = H.to_dev(lay.block_table, dev)
    lens_dev = torch.from_numpy(lay.seq_lens.copy()).to(dev)
    out = torch.full(tuple(q.shape), H.CANARY, dtype=torch.int16, device=dev)
    st = torch.cuda.current_stream().cuda_stream
    h.plan(lay.seq_lens, ws.data_ptr(), ws.numel(), st)
    h.decode_attn_multi(q.data_ptr(), q_len, k.data_ptr(), v.data_ptr(), btd.data_ptr(), lens_dev.data_ptr(),
                        out.data_ptr(), st)
    torch.cuda.synchronize()
    assert h.debug_error_word() == 0
    got_all = H.bf16_dev_to_f32(out)
    assert np.all(np.isfinite(got_all))
    WORST[(f"q_len {q_len}", name, 0)] = H.compare_every_sequence(
        got_all, q, k, v, lay.block_table, lay.seq_lens,
        lambda *a: O.paged_multi_token_attention(*a)[0], gates)
    h.close()
