"""Pins of the ring all-reduce oracle to facts it did not produce itself."""
import numpy as np
import pytest

from oracle import ring_oracle as R


def test_chunks_tile_the_vector():
    for n in (0, 1, 7, 16, 1000):
        for ranks in (1, 2, 3, 8):
            b = R.chunk_bounds(n, ranks)
            assert b[0] == 0 and b[-1] == n and len(b) == ranks + 1
            sizes = np.diff(b)
            assert np.all(sizes >= 0) and sizes.max() - sizes.min() <= 1 and np.all(np.diff(sizes) <= 0)


@pytest.mark.parametrize("ranks", [1, 2, 3, 4, 8])
def test_small_integers_sum_exactly_and_all_ranks_agree(ranks):
    rng = np.random.default_rng(ranks)
    xs = [rng.integers(-100, 101, size=1003).astype(np.float32) for _ in range(ranks)]
    want = np.sum(np.stack(xs).astype(np.int64), axis=0)
    for dtype in ("f32", "bf16"):       # |sums| <= 800 < 2^8 * ... : exact in bf16 only while below 256
        small = [np.clip(x, -30, 30) for x in xs] if dtype == "bf16" else xs
        want_d = np.sum(np.stack(small).astype(np.int64), axis=0)
        out = R.ring_all_reduce(small, dtype)
        assert len(out) == ranks
        for o in out:
            assert np.array_equal(o.astype(np.int64), want_d)


@pytest.mark.parametrize("ranks", [2, 3, 5, 8])
def test_close_to_the_float64_sum(ranks):
    rng = np.random.default_rng(10 + ranks)
    xs = [rng.standard_normal(4099).astype(np.float32) for _ in range(ranks)]
    want = np.sum(np.stack(xs).astype(np.float64), axis=0)
    out = R.ring_all_reduce(xs, "f32")
    scale = np.sum(np.abs(np.stack(xs)).astype(np.float64), axis=0)
    for o in out:
        assert np.all(np.abs(o.astype(np.float64) - want) <= (ranks - 1) * 2.0 ** -24 * scale)
        assert np.array_equal(o, out[0])


def test_one_rank_is_the_identity_and_two_ranks_are_one_addition():
    rng = np.random.default_rng(3)
    a, b = rng.standard_normal(37).astype(np.float32), rng.standard_normal(37).astype(np.float32)
    assert np.array_equal(R.ring_all_reduce([a])[0], a)
    out = R.ring_all_reduce([a, b])
    assert np.array_equal(out[0], a + b) and np.array_equal(out[1], a + b)


def test_order_of_additions_per_chunk():
    # chunk c starts at rank c and picks up ranks c+1, c+2, ... in turn: with values chosen so that float32 addition is
    # not associative, only that order gives the expected bits
    ranks, n = 4, 4
    big, tiny = np.float32(2.0 ** 24), np.float32(1.0)
    xs = [np.zeros(n, dtype=np.float32) for _ in range(ranks)]
    # chunk 0 (element 0): rank 0 holds 2^24, ranks 1..3 hold 1: ((2^24 + 1) + 1) + 1 = 2^24 in float32
    xs[0][0] = big; xs[1][0] = tiny; xs[2][0] = tiny; xs[3][0] = tiny
    # chunk 1 (element 1): starts at rank 1: ((1 + 1) + 1) + 2^24 = 2^24 + 3 -> rounds to 2^24 + 4 (ties to even)
    xs[1][1] = tiny; xs[2][1] = tiny; xs[3][1] = tiny; xs[0][1] = big
    out = R.ring_all_reduce(xs)
    assert out[0][0] == big
    assert out[0][1] == np.float32(2.0 ** 24 + 4)
    for o in out:
        assert np.array_equal(o, out[0])


def test_bf16_rounds_after_every_step():
    # 1 + 2^-8 is not a bf16 number: rounded away at once, so adding 2^-8 twice to 1 leaves 1 (ties to even), while a
    # float32 accumulation rounded once at the end would give 1 + 2^-7
    one, eps = np.float32(1.0), np.float32(2.0 ** -8)
    xs = [np.array([one], dtype=np.float32), np.array([eps], dtype=np.float32), np.array([eps], dtype=np.float32)]
    out = R.ring_all_reduce(xs, "bf16")
    assert out[0][0] == one
