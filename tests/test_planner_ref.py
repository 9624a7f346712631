"""Properties the planning rule must have, checked on the reference planner (plain integers).
The bucket facts come from the paper: degrees are powers of two like {1,2,4,8} (Section 4.3),
buckets are ordered by capacity and longer requests go to higher degrees (Sections 2.3, 4.3, 5),
work is issued longest first for the min-max objective (Section 4.3)."""
import itertools

import numpy as np
import pytest

from oracle import planner_ref as P
from paper_2606_03077_b200 import workloads as W


def check_plan(lens, hkv, params):
    pl = P.plan(lens, hkv, params)
    A = params.chunk_align
    assert pl.chunk_target % A == 0 and pl.chunk_target >= params.min_chunk
    run = 0
    for b, L in enumerate(lens):
        assert pl.item_offset[b] == run
        run += pl.num_splits[b]
        if L == 0:
            assert pl.num_splits[b] == 0 and pl.bucket[b] == -1 and pl.chunk_len[b] == 0
            continue
        s = 1 << pl.bucket[b]
        assert s <= params.max_splits and 1 <= pl.num_splits[b] <= min(s + 1, params.max_splits)   # + 1: wave fill
        assert pl.chunk_len[b] % A == 0 and pl.chunk_len[b] % 16 == 0
        # bucket bins: (C 2^(k-1), C 2^k], except that the top bucket is open-ended; with a short base chunk the
        # limits sit at the geometric means instead: [C 2^(k-1) * 181/128, C 2^k * 181/128)
        C = pl.chunk_target
        if C >= params.small_base:
            if s < params.max_splits:
                assert L <= C * s
            if s > 1:
                assert L > C * (s // 2)
        else:
            if s < params.max_splits:
                assert 128 * L < 181 * C * s
            if s > 1:
                assert 128 * L >= 181 * C * (s // 2)
        # chunks tile [0, L) exactly
        mine = sorted((it for it in pl.items if it[0] == b), key=lambda it: it[1])
        assert [it[1] for it in mine] == list(range(pl.num_splits[b]))
        pos = 0
        for (_, j, lo, hi) in mine:
            assert lo == pos and hi > lo and lo == j * pl.chunk_len[b]
            pos = hi
        assert pos == L
    assert len(pl.items) == run
    sizes = [it[3] - it[2] for it in pl.items]
    assert sizes == sorted(sizes, reverse=True)
    keys = [(-(it[3] - it[2]), it[0], it[1]) for it in pl.items]
    assert keys == sorted(keys)
    assert pl.combine == [b for b in range(len(lens)) if pl.num_splits[b] > 1]
    assert pl.empty == [b for b in range(len(lens)) if lens[b] == 0]
    # longer never gets a smaller bucket
    order = np.argsort(lens, kind="stable")
    bk = [pl.bucket[i] for i in order]
    assert bk == sorted(bk)
    check_wave_fill(lens, hkv, params, pl)
    return pl


def check_wave_fill(lens, hkv, params, pl):
    """What the wave fill may and may not do, against the same rule without it."""
    import dataclasses
    pl0 = P.plan(lens, hkv, dataclasses.replace(params, wave_fill=0))
    W_ = params.n_sm * params.ctas_per_sm
    U0 = hkv * sum(pl0.num_splits)
    k = P.cd(U0, W_)
    assert pl.chunk_target == pl0.chunk_target and pl.bucket == pl0.bucket
    if not (1 <= k <= params.wave_fill):
        assert pl == pl0
        return
    spare = (k * W_ - U0) // hkv
    assert hkv * sum(pl.num_splits) <= k * W_             # the launch does not grow into another wave
    changed = [b for b in range(len(lens)) if (pl.num_splits[b], pl.chunk_len[b]) != (pl0.num_splits[b], pl0.chunk_len[b])]
    first = sorted((b for b in range(len(lens)) if lens[b] > 0), key=lambda b: (-pl0.chunk_len[b], b))[:spare]
    assert set(changed) <= set(first)                     # only the sequences with the longest chunks
    for b in first:
        c = P.au(P.cd(lens[b], pl0.num_splits[b] + 1), params.chunk_align)
        if b in changed:
            assert c >= params.min_chunk and c < pl0.chunk_len[b] and pl0.num_splits[b] < params.max_splits
            assert pl.chunk_len[b] == c and pl.num_splits[b] == P.cd(lens[b], c)
        else:   # left alone: the shorter chunk is not allowed, or rounding made it the same chunk
            assert c < params.min_chunk or pl0.num_splits[b] >= params.max_splits or c == pl0.chunk_len[b]


def test_exhaustive_small_vectors():
    prm = P.PlanParams(n_sm=2, ctas_per_sm=1, items_per_slot=2, chunk_align=16, min_chunk=16, max_splits=4)
    n = 0
    for B in (1, 2, 3):
        for lens in itertools.product(range(0, 41, 3 if B == 3 else 1), repeat=B):
            check_plan(list(lens), 1, prm)
            n += 1
    assert n > 1000


def test_hand_worked_example():
    # n_sm 2, 1 block each, 2 items per slot, A = 16, C_min = 16, S_max = 4, one KV head
    # T = 100 + 16 + 40 = 156; C = max(16, au(cd(156, 4), 16)) = au(39, 16) = 48
    # L=100: cd(100,48)=3 -> p2 = 4; C is short and 100 * 128 = 12800 < 2 * 48 * 181 = 17376, so 2 splits (100 / 48 = 2.08
    #        is nearer to 2 than to 4); chunk = au(50,16) = 64; n = cd(100,64) = 2
    # L=16 : 1 split, chunk 16; L=40: 1 split, chunk au(40,16)=48, n = 1
    prm = P.PlanParams(n_sm=2, ctas_per_sm=1, items_per_slot=2, chunk_align=16, min_chunk=16, max_splits=4)
    pl = P.plan([100, 16, 40], 1, prm)
    assert pl.chunk_target == 48
    assert pl.bucket == [1, 0, 0] and pl.num_splits == [2, 1, 1] and pl.chunk_len == [64, 16, 48]
    assert pl.item_offset == [0, 2, 3]
    assert pl.items == [(0, 0, 0, 64), (2, 0, 0, 40), (0, 1, 64, 100), (1, 0, 0, 16)]
    # L=140 (T = 156 again): cd(140,48)=3 -> p2 = 4 and 140 * 128 = 17920 >= 17376: degree 4 stays; chunk au(35,16)=48, n = 3
    pl = P.plan([140, 16, 0], 1, prm)
    assert pl.chunk_target == 48 and pl.bucket == [2, 0, -1] and pl.num_splits == [3, 1, 0] and pl.chunk_len == [48, 16, 0]
    pl = P.plan([100, 16, 40], 1, prm)
    assert pl.combine == [0] and pl.empty == []


def test_random_vectors_default_params():
    rng = np.random.default_rng(0)
    for _ in range(200):
        B = int(rng.integers(1, 300))
        lens = np.clip(np.floor(rng.choice([64, 1024, 8192]) * np.exp(rng.normal(size=B))), 0, 40960).astype(int)
        check_plan(list(lens), int(rng.choice([1, 2, 8])), P.PlanParams())


@pytest.mark.parametrize("name,step,C,n_plain,n_items", [
    ("tiny", 0, 512, 4, 4), ("lognormal_b64", 0, 768, 158, 122), ("longtail_mix_b256", 0, 8192, 334, 334),
    ("straggler_b8", 0, 1792, 256, 128), ("shift_b128", 0, 1536, 226, 182), ("shift_b128", 1, 2560, 222, 186),
    ("shift_b128", 2, 5632, 239, 239)])
def test_workload_plans(name, step, C, n_plain, n_items):
    """With 2 x 148 slots and 4 items per slot: the item counts of the plain rule (least power of two above L / C for
    every base length) and of the rule as it stands (the nearer power of two where the base is short)."""
    lay, _ = W.make_layout(name, step)
    lens = [int(x) for x in lay.seq_lens]
    plain = P.plan(lens, lay.workload.num_kv_heads, P.PlanParams(ctas_per_sm=2, items_per_slot=4, small_base=0))
    assert plain.chunk_target == C and len(plain.items) == n_plain
    for b, L in enumerate(lens):
        s = 1 << plain.bucket[b]
        assert C * (s // 2) < L and (L <= C * s or s == 64)
    pl = check_plan(lens, lay.workload.num_kv_heads, P.PlanParams(ctas_per_sm=2, items_per_slot=4))
    assert pl.chunk_target == C and len(pl.items) == n_items
    check_plan(lens, lay.workload.num_kv_heads, P.PlanParams())


def test_straggler_split_follows_the_base_chunk():
    lay, _ = W.make_layout("straggler_b8")
    # 8 x 148 slots: base 1792 tokens, 32768 / 1792 = 18.3 is nearer to 16 than to 32 and the base is short: 16 ways
    pl = P.plan(lay.seq_lens, 8, P.PlanParams(ctas_per_sm=2, items_per_slot=4))
    assert pl.chunk_target == 1792 and set(pl.bucket) == {4} and set(pl.chunk_len) == {2048} and set(pl.num_splits) == {16}
    # 148 slots: base 14336 tokens, long chunks keep the least power of two above 32768 / 14336 = 2.3: 4 ways
    pl = P.plan(lay.seq_lens, 8, P.PlanParams(wave_fill=0))
    assert pl.chunk_target == 14336 and set(pl.bucket) == {2} and set(pl.chunk_len) == {8192} and set(pl.num_splits) == {4}
    # that is 8 * 4 * 8 = 256 blocks on 148 slots: 1.73 waves.  The 40 free slots of the second wave are 5 work items:
    # the first five sequences are cut 5 ways, chunk au(cd(32768, 5), 256) = 6656 -> 37 items = 296 blocks = 2 full waves
    pl = P.plan(lay.seq_lens, 8, P.PlanParams())
    assert pl.chunk_target == 14336 and set(pl.bucket) == {2}
    assert pl.num_splits == [5] * 5 + [4] * 3 and pl.chunk_len == [6656] * 5 + [8192] * 3
    assert len(pl.items) * 8 == 2 * 148
    assert [it[3] - it[2] for it in pl.items] == [8192] * 12 + [6656] * 20 + [6144] * 5


def test_wave_fill_hand_worked():
    # one wave: 4 slots, one KV head, A = 16, C_min = 16.  T = 288, C = au(cd(288, 4), 16) = 80; every 96 is one chunk
    # (cd(96, 80) = 2 -> p2 = 2, but C is short and 96 * 128 = 12288 < 1 * 80 * 181 = 14480: 1).  3 blocks on 4 slots:
    # 1 free slot -> the first sequence (equal chunks: lowest index) is cut in two, chunk au(cd(96, 2), 16) = 48
    prm = P.PlanParams(n_sm=4, ctas_per_sm=1, items_per_slot=1, chunk_align=16, min_chunk=16, max_splits=8)
    pl = P.plan([96, 96, 96], 1, prm)
    assert pl.chunk_target == 80 and pl.bucket == [0, 0, 0]
    assert pl.num_splits == [2, 1, 1] and pl.chunk_len == [48, 96, 96] and pl.item_offset == [0, 2, 3]
    assert pl.items == [(1, 0, 0, 96), (2, 0, 0, 96), (0, 0, 0, 48), (0, 1, 48, 96)] and pl.combine == [0]
    # two waves: 3 slots, four sequences of 64.  T = 256, C = au(cd(256, 3), 16) = 96, one chunk each: 4 blocks = 2 waves
    # with 2 free slots -> sequences 0 and 1 are cut in two (chunk 32)
    prm = P.PlanParams(n_sm=3, ctas_per_sm=1, items_per_slot=1, chunk_align=16, min_chunk=16, max_splits=8)
    pl = P.plan([64, 64, 64, 64], 1, prm)
    assert pl.chunk_target == 96 and pl.num_splits == [2, 2, 1, 1] and pl.chunk_len == [32, 32, 64, 64]
    assert pl.items == [(2, 0, 0, 64), (3, 0, 0, 64), (0, 0, 0, 32), (0, 1, 32, 64), (1, 0, 0, 32), (1, 1, 32, 64)]
    # two KV heads: every work item is two blocks.  [64] * 4 on 5 slots: T = 256, C = au(cd(512, 5), 16) = 112; 8 blocks
    # = 2 waves of 5 with 2 free slots = 1 item -> only sequence 0 is cut
    prm = P.PlanParams(n_sm=5, ctas_per_sm=1, items_per_slot=1, chunk_align=16, min_chunk=16, max_splits=8)
    pl = P.plan([64, 64, 64, 64], 2, prm)
    assert pl.chunk_target == 112 and pl.num_splits == [2, 1, 1, 1] and pl.chunk_len == [32, 64, 64, 64]
    # three waves and more: left alone (wave_fill = 2)
    prm = P.PlanParams(n_sm=2, ctas_per_sm=1, items_per_slot=1, chunk_align=16, min_chunk=16, max_splits=8)
    pl = P.plan([64, 64, 64, 64, 64], 1, prm)
    assert pl.num_splits == [1] * 5
    # a chunk below C_min is not made: 1 wave of 4 slots, lengths 16: nothing to cut
    prm = P.PlanParams(n_sm=4, ctas_per_sm=1, items_per_slot=1, chunk_align=16, min_chunk=16, max_splits=8)
    assert P.plan([16, 16], 1, prm).num_splits == [1, 1]
