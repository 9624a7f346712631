"""Pins of the KV-migration oracle: identities that hold for any correct rearrangement (round trip,
split-then-concatenate, head ranges compose), and one hand-written tiny case."""
import numpy as np

from oracle import kv_move_oracle as M
from paper_2606_03077_b200 import workloads as W


def case(seed=0, lens=(1, 17, 40), hkv=4, d=8):
    rng = np.random.default_rng(seed)
    lens = np.asarray(lens, np.int32)
    bt, pool = W.draw_block_table(lens, int(W.pages_needed(lens).sum()) + 3, rng)
    pages = rng.integers(0, 65536, (pool, hkv, 16, d)).astype(np.uint16)
    return lens, bt, pages


def test_hand_written_case():
    # two pages of one head, d = 2: token t of the sequence holds (100 t, 100 t + 1)
    pages = np.zeros((3, 1, 16, 2), np.uint16)
    bt = np.array([[2, 0]], np.int32)
    for t in range(20):
        pages[bt[0, t // 16], 0, t % 16] = (100 * t, 100 * t + 1)
    dense = M.gather(pages, bt, [20], 0, 1)
    assert dense.shape == (20, 1, 2)
    assert [int(x) for x in dense[:, 0, 0]] == [100 * t for t in range(20)]
    assert int(dense[19, 0, 1]) == 1901 and int(dense[16, 0, 0]) == 1600   # token 16 is slot 0 of page 0


def test_round_trip_and_head_ranges():
    lens, bt, pages = case()
    full = M.gather(pages, bt, lens, 0, 4)
    assert full.shape == (int(lens.sum()), 4, 8)
    # a head range of the pool is the same head range of the full gather
    assert np.array_equal(M.gather(pages, bt, lens, 1, 2), full[:, 1:3])
    # split then concatenate restores the partition
    assert np.array_equal(M.concat_heads(M.split_heads(full, 2)), full)
    assert np.array_equal(M.concat_heads(M.split_heads(full, 4)), full)
    # scatter into a fresh pool with another placement, gather again: identical
    rng = np.random.default_rng(9)
    bt2, pool2 = W.draw_block_table(lens, int(W.pages_needed(lens).sum()) + 7, rng)
    fresh = np.full((pool2, 4, 16, 8), 0xFFFF, np.uint16)
    M.scatter(full, fresh, bt2, lens, 0)
    assert np.array_equal(M.gather(fresh, bt2, lens, 0, 4), full)
    # slots past the end were not written
    last = bt2[1, (17 - 1) // 16]
    assert np.all(fresh[last, :, 1:, :] == 0xFFFF)


def test_tp_reshard_composes():
    # TP 1 -> TP 2: two shards land in two pools of 2 heads each; TP 2 -> TP 1 concatenates them back
    lens, bt, pages = case(seed=2)
    shards = M.split_heads(M.gather(pages, bt, lens, 0, 4), 2)
    pools = [np.zeros((pages.shape[0], 2, 16, 8), np.uint16) for _ in range(2)]
    for r in range(2):
        M.scatter(shards[r], pools[r], bt, lens, 0)
        assert np.array_equal(M.gather(pools[r], bt, lens, 0, 2), M.gather(pages, bt, lens, 2 * r, 2))
    back = np.zeros_like(pages)
    for r in range(2):
        M.scatter(M.gather(pools[r], bt, lens, 0, 2), back, bt, lens, 2 * r)
    assert np.array_equal(M.gather(back, bt, lens, 0, 4), M.gather(pages, bt, lens, 0, 4))
