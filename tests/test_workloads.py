"""The seeded generators: recipes reproduce their documented check values and the long-tail shape
the paper reports (Section 2.2: the longest 10 % of trajectories take over half of rollout time)."""
import numpy as np

from paper_2606_03077_b200 import workloads as W


def test_bf16_round_to_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, 1.0 + 2 ** -9], dtype=np.float32)  # ties at 2^-8 steps
    b = W.f32_to_bf16_bits(x)
    assert list(b) == [0x3F80, 0x3F80, 0x3F82, 0x3F80]
    assert np.array_equal(W.bf16_bits_to_f32(b), np.array([1.0, 1.0, 1.015625, 1.0], dtype=np.float32))


def test_check_values():
    lay, _ = W.make_layout("tiny")
    assert list(lay.seq_lens) == [1, 7, 64, 300] and lay.pool_pages == 64
    assert list(lay.block_table[0, :1]) == [16] and list(lay.block_table[1, :1]) == [36]
    assert list(lay.block_table[2, :3]) == [27, 8, 44] and lay.kv_bytes == 95232
    lay, _ = W.make_layout("lognormal_b64")
    assert lay.total_tokens == 89875 and list(lay.seq_lens[:3]) == [1132, 921, 1709]
    assert int(W.pages_needed(lay.seq_lens).sum()) == 5646 and lay.seq_lens.max() == 4913
    lay, _ = W.make_layout("longtail_mix_b256")
    assert lay.total_tokens == 1177146 and lay.seq_lens.max() == 32212
    assert int((lay.seq_lens >= 16384).sum()) == 26
    top = np.sort(lay.seq_lens.astype(np.int64))[::-1][:26].sum() / lay.total_tokens
    assert top > 0.5  # the 10 % tail holds more than half of the work
    lay, _ = W.make_layout("straggler_b8")
    assert lay.kv_bytes == 1073741824
    for st, tok in enumerate((212788, 370435, 821788)):
        lay, _ = W.make_layout("shift_b128", st)
        assert lay.total_tokens == tok and lay.pool_pages == 262144


def test_block_tables_are_disjoint_and_in_range():
    for name in ("tiny", "lognormal_b64", "shift_b128"):
        lay, _ = W.make_layout(name)
        used = lay.block_table[lay.block_table >= 0]
        assert len(used) == int(W.pages_needed(lay.seq_lens).sum())
        assert len(np.unique(used)) == len(used) and used.max() < lay.pool_pages
        for b, L in enumerate(lay.seq_lens):
            n = (int(L) + 15) // 16
            assert np.all(lay.block_table[b, :n] >= 0) and np.all(lay.block_table[b, n:] == -1)


def test_host_inputs_poisoned_outside():
    lay, q, k, v = W.make_host_inputs("tiny")
    kf = W.bf16_bits_to_f32(k)
    owned = np.zeros(k.shape[0] * 16, dtype=bool).reshape(-1, 16)
    for b, L in enumerate(lay.seq_lens):
        for t in range(int(L)):
            owned[lay.block_table[b, t // 16], t % 16] = True
    assert np.all(np.abs(kf[:, 0][owned]) <= 1.0)
    assert np.all(kf[:, 0][~owned] > 1e29)
    assert np.all(np.abs(W.bf16_bits_to_f32(q)) <= 1.0)


def test_e4m3_case_generator():
    # codes are made from bit fields: live slots are finite with exponent field <= 8, dead slots hold the NaN code
    lens, bt, q, k8, v8 = W.random_case_e4m3(5, 3, 4, 2, 16, (3, 16, 21))
    lens2, bt2, q2, k82, v82 = W.random_case_e4m3(5, 3, 4, 2, 16, (3, 16, 21))
    assert np.array_equal(k8, k82) and np.array_equal(v8, v82) and np.array_equal(bt, bt2) and np.array_equal(q, q2)
    assert k8.dtype == np.uint8 and k8.shape == v8.shape and k8.shape[1:] == (2, 16, 16)
    live = np.zeros(k8.shape[0] * 16, dtype=bool).reshape(-1, 16)
    for b, L in enumerate(lens):
        for t in range(int(L)):
            live[bt[b, t // 16], t % 16] = True
    for pool, nan in ((k8, W.E4M3_NAN), (v8, W.E4M3_NAN | 0x80)):
        lv = pool.transpose(0, 2, 1, 3)[live]
        assert np.all(((lv >> 3) & 0xF) <= 8)
        assert np.all(pool.transpose(0, 2, 1, 3)[~live] == nan)
    assert len(np.unique(bt[bt >= 0])) == int(W.pages_needed(lens).sum())
