"""Pins of the CPU oracle to facts it did not produce itself: special cases, closed forms,
invariants, a loop-only brute force.  A dropped term, wrong sign, wrong scale, wrong head map,
transposed operand or off-by-one gather fails at least one of them.  The paper prints no worked
example for attention, so there are no paper values to pin against."""
import math

import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W

import gates


def bits(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def small_case(seed=3, B=3, Hq=4, Hkv=2, d=16, lens=(1, 17, 40)):
    return W.random_case(seed, B, Hq, Hkv, d, lens, values="normal")


def dense_rows(pages, bt_row, L, head):
    """Independent gather with explicit indexing (HND)."""
    return [W.bf16_bits_to_f32(pages[bt_row[t // 16], head, t % 16]).astype(np.float64) for t in range(L)]


def test_bf16_conversion_is_exact():
    vals = np.array([0.0, 1.0, -2.5, 0.1, 3.0e-5, 1e30, -1e-30], dtype=np.float32)
    b = bits(vals)
    back = O.bf16_bits_to_f64(b)
    assert np.array_equal(back, W.bf16_bits_to_f32(b).astype(np.float64))
    # 1.0 is 0x3F80, -2.5 is 0xC020 in bf16
    assert b[1] == 0x3F80 and b[2] == 0xC020
    assert back[1] == 1.0 and back[2] == -2.5


def test_length_one_returns_v0():
    lens, bt, q, k, v = W.random_case(5, 2, 4, 2, 16, (1, 1))
    out, lse = O.paged_decode_attention(q, k, v, bt, lens)
    for b in range(2):
        for h in range(4):
            v0 = W.bf16_bits_to_f32(v[bt[b, 0], h // 2, 0]).astype(np.float64)
            assert np.array_equal(out[b, h], v0)
            k0 = W.bf16_bits_to_f32(k[bt[b, 0], h // 2, 0]).astype(np.float64)
            qq = W.bf16_bits_to_f32(q[b, h]).astype(np.float64)
            assert lse[b, h] == pytest.approx(float(qq @ k0) / 4.0, rel=1e-14)


def test_identical_value_rows_return_that_row():
    lens, bt, q, k, v = small_case()
    row = bits(np.linspace(-2, 2, 16))
    v[...] = row
    out, _ = O.paged_decode_attention(q, k, v, bt, lens)
    assert np.allclose(out, O.bf16_bits_to_f64(row), rtol=0, atol=1e-14)


def test_zero_query_gives_mean_closed_form():
    # v_t[j] = (t + j) mod 251, exact in bf16 (< 256); mean over t is a rational number
    L = 75
    lens, bt, q, k, v = W.random_case(7, 1, 2, 1, 16, (L,))
    q[...] = 0
    for t in range(L):
        v[bt[0, t // 16], 0, t % 16] = bits([(t + j) % 251 for j in range(16)])
    out, lse = O.paged_decode_attention(q, k, v, bt, lens)
    for j in range(16):
        exact = sum((t + j) % 251 for t in range(L)) / L
        assert out[0, 0, j] == pytest.approx(exact, rel=1e-14)
        assert out[0, 1, j] == pytest.approx(exact, rel=1e-14)
    assert lse[0, 0] == pytest.approx(math.log(L), rel=1e-14)


def test_identical_keys_give_mean():
    L = 33
    lens, bt, q, k, v = W.random_case(8, 1, 2, 1, 16, (L,))
    k[...] = bits(np.arange(16) / 8.0)
    out, _ = O.paged_decode_attention(q, k, v, bt, lens)
    rows = np.array(dense_rows(v, bt[0], L, 0))
    assert np.allclose(out[0, 0], rows.mean(axis=0), rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("tstar", [0, 15, 16, 31, 32, 36])
def test_one_hot_key_selects_its_value_row(tstar):
    L, d = 37, 16
    lens, bt, q, k, v = W.random_case(9, 1, 2, 1, d, (L,))
    c = 32.0  # score gap c*c/sqrt(d) = 256: every other weight is e^-256, far below float64 resolution
    k[...] = 0
    q[...] = 0
    q[0, :, 0] = bits([c])[0]
    k[bt[0, tstar // 16], 0, tstar % 16, 0] = bits([c])[0]
    # a dominant key just past the end must have no effect
    k[bt[0, L // 16], 0, L % 16, 0] = bits([4 * c])[0]
    out, _ = O.paged_decode_attention(q, k, v, bt, lens)
    want = W.bf16_bits_to_f32(v[bt[0, tstar // 16], 0, tstar % 16]).astype(np.float64)
    # the other L-1 weights are e^-256 each: far below float64 resolution of the result
    assert np.allclose(out[0, 0], want, rtol=1e-15, atol=1e-100)
    assert np.array_equal(O.round_to_bf16(out[0, 1]), want)


def test_two_token_logistic_closed_form():
    # softmax over two scores is a logistic: out = sig(D) v0 + (1 - sig(D)) v1, D = (q.k0 - q.k1) * scale
    d = 16
    lens, bt, q, k, v = W.random_case(10, 1, 1, 1, d, (2,))
    qq = O.bf16_bits_to_f64(q[0, 0])
    k0, k1 = (O.bf16_bits_to_f64(k[bt[0, 0], 0, i]) for i in (0, 1))
    v0, v1 = (O.bf16_bits_to_f64(v[bt[0, 0], 0, i]) for i in (0, 1))
    D = (float(qq @ k0) - float(qq @ k1)) / math.sqrt(d)
    sig = 1.0 / (1.0 + math.exp(-D))
    out, lse = O.paged_decode_attention(q, k, v, bt, lens)
    assert np.allclose(out[0, 0], sig * v0 + (1 - sig) * v1, rtol=1e-13, atol=1e-14)
    assert lse[0, 0] == pytest.approx(float(qq @ k0) / 4 + math.log1p(math.exp(-D)), rel=1e-13)
    # explicit scale overrides the default
    out2, _ = O.paged_decode_attention(q, k, v, bt, lens, sm_scale=0.5)
    sig2 = 1.0 / (1.0 + math.exp(-(float(qq @ k0) - float(qq @ k1)) * 0.5))
    assert np.allclose(out2[0, 0], sig2 * v0 + (1 - sig2) * v1, rtol=1e-13, atol=1e-14)


def test_gqa_head_map_is_contiguous_groups():
    # value rows of KV head g are the constant g + 1, so query head h must return h // G + 1
    lens, bt, q, k, v = W.random_case(11, 2, 8, 4, 16, (20, 5))
    for g in range(4):
        v[:, g] = bits([g + 1.0])[0]
    out, _ = O.paged_decode_attention(q, k, v, bt, lens)
    for h in range(8):
        assert np.allclose(out[:, h], h // 2 + 1.0, atol=1e-14)


def test_page_placement_does_not_matter():
    lens, bt, q, k, v = small_case(seed=12)
    out, lse = O.paged_decode_attention(q, k, v, bt, lens)
    rng = np.random.default_rng(1)
    perm = rng.permutation(k.shape[0])           # new id of old page i is perm[i]
    k2 = np.empty_like(k); v2 = np.empty_like(v)
    k2[perm] = k; v2[perm] = v
    bt2 = np.where(bt >= 0, perm[np.maximum(bt, 0)], -1).astype(np.int32)
    out2, lse2 = O.paged_decode_attention(q, k2, v2, bt2, lens)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_nhd_layout_equals_hnd():
    lens, bt, q, k, v = small_case(seed=13)
    out, lse = O.paged_decode_attention(q, k, v, bt, lens)
    kn = np.ascontiguousarray(k.transpose(0, 2, 1, 3)); vn = np.ascontiguousarray(v.transpose(0, 2, 1, 3))
    out2, lse2 = O.paged_decode_attention(q, kn, vn, bt, lens, layout="NHD")
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_dense_loop_brute_force_agrees():
    lens, bt, q, k, v = small_case(seed=14, B=3, Hq=4, Hkv=2, d=8, lens=(1, 19, 33))
    out, lse = O.paged_decode_attention(q, k, v, bt, lens)
    for b in range(3):
        for h in range(4):
            K = dense_rows(k, bt[b], int(lens[b]), h // 2)
            V = dense_rows(v, bt[b], int(lens[b]), h // 2)
            o, l = O.dense_attention_loops(W.bf16_bits_to_f32(q[b, h]).astype(np.float64), K, V, 1 / math.sqrt(8))
            assert np.max(np.abs(out[b, h] - np.array(o))) <= 1e-12
            assert abs(lse[b, h] - l) <= 1e-12


def test_tiny_workload_against_brute_force():
    lay, q, k, v = W.make_host_inputs("tiny")
    out, lse = O.paged_decode_attention(q, k, v, lay.block_table, lay.seq_lens)
    for b in range(4):
        for h in (0, 3):
            L = int(lay.seq_lens[b])
            K = dense_rows(k, lay.block_table[b], L, 0)
            V = dense_rows(v, lay.block_table[b], L, 0)
            o, l = O.dense_attention_loops(W.bf16_bits_to_f32(q[b, h]).astype(np.float64), K, V, 0.125)
            assert np.max(np.abs(out[b, h] - np.array(o))) <= 1e-12
            assert abs(lse[b, h] - l) <= 1e-12


@pytest.mark.parametrize("shift", [80.0, -200.0])
def test_key_shift_only_moves_the_scores(shift):
    # adding u to every key adds q.u*scale to every score: out unchanged, lse moves by that amount
    lens, bt, q, k, v = small_case(seed=15)
    out, lse = O.paged_decode_attention(q, k, v, bt, lens)
    u = np.zeros(16); u[0] = shift
    kf = W.bf16_bits_to_f32(k).astype(np.float64) + u
    k2 = bits(kf)
    # the shifted keys must still be exact bf16 values for the identity to be exact: rebuild the
    # unshifted keys from the rounded shifted ones
    k1 = bits(W.bf16_bits_to_f32(k2).astype(np.float64) - u)
    assert np.array_equal(W.bf16_bits_to_f32(k1).astype(np.float64) + u, W.bf16_bits_to_f32(k2).astype(np.float64))
    out1, lse1 = O.paged_decode_attention(q, k1, v, bt, lens)
    out2, lse2 = O.paged_decode_attention(q, k2, v, bt, lens)
    q0 = O.bf16_bits_to_f64(q)[:, :, 0]
    assert np.allclose(out1, out2, rtol=1e-9, atol=1e-11)
    assert np.allclose(lse2 - lse1, q0 * shift / 4.0, rtol=1e-9, atol=1e-9)


def test_chunked_merge_equals_direct():
    L = 100
    lens, bt, q, k, v = W.random_case(16, 1, 2, 1, 16, (L,))
    out, lse = O.paged_decode_attention(q, k, v, bt, lens)
    # evaluate [0,32), [32,80), [80,100) as separate "sequences" sharing the pages, then merge
    cuts = [(0, 32), (32, 80), (80, 100)]
    parts_o, parts_l = [], []
    for a, e in cuts:
        bt_c = bt[:, a // 16:]
        o, l = O.paged_decode_attention(q, k, v, bt_c, np.array([e - a], dtype=np.int32))
        parts_o.append(o[0]); parts_l.append(l[0])
    for h in range(2):
        mo, ml = O.merge_partials([p[h] for p in parts_o], [p[h] for p in parts_l])
        assert np.max(np.abs(mo - out[0, h])) <= 1e-12
        assert abs(ml - lse[0, h]) <= 1e-12


def test_empty_sequence_is_zero():
    lens, bt, q, k, v = W.random_case(17, 2, 2, 1, 16, (0, 3))
    out, lse = O.paged_decode_attention(q, k, v, bt, lens)
    assert np.all(out[0] == 0) and np.all(np.isneginf(lse[0]))
    assert np.all(np.isfinite(out[1]))


def test_poison_outside_sequences_is_never_read():
    lens, bt, q, k, v = W.random_case(18, 2, 2, 1, 16, (5, 21), poison=True)
    lens2, bt2, q2, k2, v2 = W.random_case(18, 2, 2, 1, 16, (5, 21), poison=False)
    a, _ = O.paged_decode_attention(q, k, v, bt, lens)
    b, _ = O.paged_decode_attention(q2, k2, v2, bt2, lens2)
    assert np.array_equal(a, b)
    assert np.max(np.abs(a)) < 10


# ----- the harness itself must notice the classic bugs (mutations of a correct result)
def test_gates_catch_mutations():
    lens, bt, q, k, v = W.random_case(19, 2, 8, 2, 64, (2048 + 5, 700))
    ref, _ = O.paged_decode_attention(q, k, v, bt, lens)
    assert gates.tight_violations(ref, ref) == 0
    # (i) a dropped 256-token chunk at the end of sequence 0
    cut = lens.copy(); cut[0] -= 256
    bad, _ = O.paged_decode_attention(q, k, v, bt, cut)
    assert gates.tight_violations(bad, ref) > 0
    # (ii) seq_len off by one
    for dl in (-1,):
        m = lens.copy(); m[1] += dl
        bad, _ = O.paged_decode_attention(q, k, v, bt, m)
        assert gates.tight_violations(bad, ref) > 0
    # (iii) two block-table entries of different sequences swapped
    bt2 = bt.copy(); bt2[0, 3], bt2[1, 2] = bt[1, 2], bt[0, 3]
    bad, _ = O.paged_decode_attention(q, k, v, bt2, lens)
    assert gates.tight_violations(bad, ref) > 0
    # (iv) head map h mod Hkv instead of h // G
    qperm = q.reshape(2, 2, 4, 64).transpose(0, 2, 1, 3).reshape(2, 8, 64)
    bad, _ = O.paged_decode_attention(np.ascontiguousarray(qperm), k, v, bt, lens)
    bad = bad.reshape(2, 2, 4, 64).transpose(0, 2, 1, 3).reshape(2, 8, 64)
    assert gates.tight_violations(bad, ref) > 0
    # (v) all zeros
    assert gates.tight_violations(np.zeros_like(ref), ref) > 0
    # bf16 rounding of a correct result passes both gates
    assert gates.tight_violations(O.round_to_bf16(ref), ref) == 0
    assert gates.stated_violations(O.round_to_bf16(ref), ref) == 0


def test_tiny_workload_matches_stored_oracle_values():
    """Regression pin: the stored values were written by tests/golden/make_tiny_golden.py from this
    oracle; a change of its arithmetic shows up here and has to be justified."""
    import os
    lay, q, k, v = W.make_host_inputs("tiny")
    out, lse = O.paged_decode_attention(q, k, v, lay.block_table, lay.seq_lens)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "tiny_expected.txt")
    n = 0
    for line in open(path):
        if line.startswith("#"):
            continue
        f = line.split()
        b, h = int(f[0]), int(f[1])
        want = [float(x) for x in f[2:]]
        got = [lse[b, h]] + [out[b, h, j] for j in (0, 21, 42, 63)]
        assert np.allclose(got, want, rtol=1e-13, atol=1e-15)
        n += 1
    assert n == 16
