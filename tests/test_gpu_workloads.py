"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times: the four
large workloads with pools filled on the device, compared with the oracle on every sequence where
that takes seconds and on a sample of sequences (longest, shortest, random) elsewhere."""
import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W

import gates
import gpu_harness as H

pytestmark = pytest.mark.gpu


def sample_rows(lens, n, seed):
    order = np.argsort(lens)
    pick = set(order[:2].tolist()) | set(order[-3:].tolist())
    rng = np.random.default_rng(seed)
    pick |= set(rng.choice(len(lens), size=min(n, len(lens)), replace=False).tolist())
    return sorted(pick)


@pytest.mark.parametrize("name,n_sample", [("lognormal_b64", 64), ("longtail_mix_b256", 24), ("straggler_b8", 2),
                                           ("shift_b128", 12)])
def test_workload_parity(lib, name, n_sample):
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
        rows = sample_rows(lay.seq_lens, n_sample, step)
        kh, vh, bth, lh = H.gather_for_oracle(k, v, bt, lay.seq_lens, rows)
        qh = q.view(torch.int16)[torch.tensor(rows, device=dev)].cpu().numpy().view(np.uint16)
        ref, _ = O.paged_decode_attention(qh, kh, vh, bth, lh)
        got = out[rows]
        assert gates.stated_violations(got, ref) == 0
        assert gates.tight_violations(got, ref) == 0, gates.tight_ratio(got, ref)
        # property that holds for every sequence: |out| <= max |v| over the pool (a convex combination)
        assert np.max(np.abs(out)) <= 6.5
        for mode in (0, 1):           # step C as its own kernel / inside the decode kernel: same bits
            r.h.set_combine_mode(mode)
            out2 = H.bf16_dev_to_f32(r.run(q, k, v, H.to_dev(bt, dev), lay.seq_lens))
            assert np.array_equal(out, out2)
        r.h.set_combine_mode(1)
        W.restore_tails(saved, k, v)
    r.h.close()
