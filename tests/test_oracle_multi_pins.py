"""Pins of the several-query-token oracle (oracle.attention_oracle.paged_multi_token_attention) to facts it did
not produce itself.  What is new relative to the single-token definition is only each query token's causal
limit n_i = L - Tq + 1 + i; every pin below fails if that limit is off by one in either direction, if rows
are attributed to the wrong query token, or if a short sequence is mishandled."""
import math

import numpy as np
import pytest

from oracle import attention_oracle as O
from paper_2606_03077_b200 import workloads as W


def bits(x):
    return W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def draw_q(seed, B, Tq, Hq, d):
    rng = np.random.default_rng(seed)
    return bits(rng.standard_normal((B, Tq, Hq, d)).astype(np.float32))


def dense_rows(pages, bt_row, L, head):
    return [W.bf16_bits_to_f32(pages[bt_row[t // 16], head, t % 16]).astype(np.float64) for t in range(L)]


def test_one_query_token_is_the_single_token_definition():
    lens, bt, q, k, v = W.random_case(11, 3, 4, 2, 16, (1, 17, 40))
    out1, lse1 = O.paged_decode_attention(q, k, v, bt, lens)
    outm, lsem = O.paged_multi_token_attention(q[:, None], k, v, bt, lens)
    assert np.array_equal(outm[:, 0], out1) and np.array_equal(lsem[:, 0], lse1)


@pytest.mark.parametrize("Tq", [2, 3, 5])
def test_each_row_is_single_token_decode_at_its_own_length(Tq):
    # query token i sees exactly what a one-token decode step would have seen when the sequence had L - Tq + 1 + i tokens
    lens, bt, _, k, v = W.random_case(12, 4, 6, 2, 16, (5, 16, 33, 70))
    q = draw_q(13, 4, Tq, 6, 16)
    outm, lsem = O.paged_multi_token_attention(q, k, v, bt, lens)
    for i in range(Tq):
        ref, lse = O.paged_decode_attention(q[:, i], k, v, bt, lens - Tq + 1 + i)
        assert np.allclose(outm[:, i], ref, rtol=0, atol=1e-13)
        assert np.allclose(lsem[:, i], lse, rtol=0, atol=1e-12)


def test_loop_brute_force_agrees():
    Tq = 3
    lens, bt, _, k, v = W.random_case(14, 2, 4, 2, 8, (4, 21))
    q = draw_q(15, 2, Tq, 4, 8)
    outm, lsem = O.paged_multi_token_attention(q, k, v, bt, lens)
    for b in range(2):
        for i in range(Tq):
            n = int(lens[b]) - Tq + 1 + i
            for h in range(4):
                K = dense_rows(k, bt[b], n, h // 2)
                V = dense_rows(v, bt[b], n, h // 2)
                o, l = O.dense_attention_loops(W.bf16_bits_to_f32(q[b, i, h]).astype(np.float64), K, V, 1 / math.sqrt(8))
                assert np.allclose(outm[b, i, h], o, rtol=0, atol=1e-12)
                assert abs(lsem[b, i, h] - l) < 1e-12


def test_zero_query_gives_the_running_mean_in_closed_form():
    # q = 0: uniform softmax, so row i is the mean of the first n_i value rows; v_t[j] = t + j gives
    # mean = (n_i - 1) / 2 + j exactly
    Tq, L, d = 4, 37, 8
    lens, bt, _, k, v = W.random_case(16, 1, 2, 1, d, (L,))
    for t in range(L):
        v[bt[0, t // 16], 0, t % 16] = bits(np.arange(d) + t)
    q = np.zeros((1, Tq, 2, d), dtype=np.uint16)
    out, lse = O.paged_multi_token_attention(q, k, v, bt, lens)
    for i in range(Tq):
        n = L - Tq + 1 + i
        assert np.allclose(out[0, i, 0], (n - 1) / 2 + np.arange(d), rtol=0, atol=1e-12)
        assert abs(lse[0, i, 1] - math.log(n)) < 1e-12


@pytest.mark.parametrize("L", [6, 16, 17, 48])
def test_one_hot_keys_on_either_side_of_every_causal_limit(L):
    # token t has key c*e_0 iff t is one of the last Tq tokens or token 0; all queries are c*e_0 with c^2*scale = 200.
    # Query token i sees the dominant keys at 0 and at the new tokens up to itself, all with the same score, so its
    # output is the plain mean of those value rows, and no later token may leak in.
    Tq, d = 4, 16
    c = math.sqrt(200.0 * math.sqrt(d))
    lens, bt, _, k, v = W.random_case(17, 1, 1, 1, d, (L,))
    rng = np.random.default_rng(18)
    vals = rng.integers(-8, 9, size=(L, d)).astype(np.float32)
    new = list(range(L - Tq, L))
    for t in range(L):
        row = np.zeros(d, dtype=np.float32)
        if t == 0 or t in new:
            row[0] = c
        k[bt[0, t // 16], 0, t % 16] = bits(row)
        v[bt[0, t // 16], 0, t % 16] = bits(vals[t])
    qrow = np.zeros(d, dtype=np.float32)
    qrow[0] = c
    q = np.broadcast_to(bits(qrow), (1, Tq, 1, d)).copy()
    out, _ = O.paged_multi_token_attention(q, k, v, bt, lens)
    cq = float(W.bf16_bits_to_f32(bits([c]))[0])
    for i in range(Tq):
        seen = sorted({0} | set(new[: i + 1]))
        want = vals[seen].astype(np.float64).mean(axis=0)
        # the other tokens have score 0 against a dominant score of cq^2 / 4 >= 190: weight < e^-190
        assert cq * cq / math.sqrt(d) > 190
        assert np.allclose(out[0, i, 0], want, rtol=0, atol=1e-60 + 1e-12)


def test_sequences_shorter_than_the_query_block():
    # L = 2 with Tq = 4: query tokens 0 and 1 have nothing to attend to (n_i <= 0): zero output, lse = -inf;
    # token 2 sees one cached token and returns its value row; token 3 sees both
    Tq, d = 4, 8
    lens, bt, _, k, v = W.random_case(19, 2, 2, 1, d, (2, 0))
    q = draw_q(20, 2, Tq, 2, d)
    out, lse = O.paged_multi_token_attention(q, k, v, bt, lens)
    assert np.all(out[0, :2] == 0) and np.all(np.isneginf(lse[0, :2]))
    v0 = W.bf16_bits_to_f32(v[bt[0, 0], 0, 0]).astype(np.float64)
    assert np.allclose(out[0, 2, 0], v0, rtol=0, atol=1e-15) and np.allclose(out[0, 2, 1], v0, rtol=0, atol=1e-15)
    assert np.all(np.isfinite(lse[0, 2:]))
    assert np.all(out[1] == 0) and np.all(np.isneginf(lse[1]))
