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
        assert 1 <= pl.num_splits[b] <= s <= params.max_splits
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
    check_refine(lens, hkv, params, pl)
    return pl


def check_refine(lens, hkv, params, pl):
    """The second pass: made exactly when the first plan is coarse (fewer than 1.5 waves) on a long base, and then it is
    the plain plan for twice as many slots."""
    import dataclasses
    pl0 = P.plan(lens, hkv, dataclasses.replace(params, refine=0))
    W_ = params.n_sm * params.ctas_per_sm
    coarse = pl0.chunk_target >= 4096 and 2 * hkv * len(pl0.items) < 3 * W_
    if not (params.refine and coarse):
        assert pl == pl0
        return
    twice = P.plan(lens, hkv, dataclasses.replace(params, refine=0, items_per_slot=2 * params.items_per_slot))
    assert pl == twice and pl.chunk_target <= pl0.chunk_target and len(pl.items) >= len(pl0.items)


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
    # 148 slots: base 14336 tokens, long chunks keep the least power of two above 32768 / 14336 = 2.3: 4 ways;
    # 8 * 4 * 8 = 256 blocks are 1.73 waves, not fewer than 1.5: the plan stands
    pl = P.plan(lay.seq_lens, 8, P.PlanParams())
    assert pl.chunk_target == 14336 and set(pl.bucket) == {2} and set(pl.chunk_len) == {8192} and set(pl.num_splits) == {4}


def test_coarse_plans_are_cut_finer_hand_worked():
    # 12 sequences of 20,000 tokens, 8 KV heads, 148 slots.  T = 240,000; C = au(cd(1,920,000, 148), 256) = au(12973, 256)
    # = 13056; cd(20000, 13056) = 2 -> 2 chunks of au(10000, 256) = 10240: 24 items = 192 blocks, and 2 * 192 = 384 < 3 * 148
    # = 444: fewer than one and a half waves, on a base >= 4096 -> again for 296 slots: C = au(cd(1,920,000, 296), 256) =
    # au(6487, 256) = 6656; cd(20000, 6656) = 4 -> 4 chunks of au(5000, 256) = 5120: 48 items = 384 blocks
    pl = P.plan([20000] * 12, 8, P.PlanParams())
    assert pl.chunk_target == 6656 and pl.bucket == [2] * 12 and pl.num_splits == [4] * 12 and pl.chunk_len == [5120] * 12
    assert [it[3] - it[2] for it in pl.items] == [5120] * 36 + [4640] * 12
    plain = P.plan([20000] * 12, 8, P.PlanParams(refine=0))
    assert plain.chunk_target == 13056 and plain.num_splits == [2] * 12 and plain.chunk_len == [10240] * 12
    # 3 sequences of 40,000: C = au(cd(960,000, 148), 256) = 6656, 8 chunks of 5120 each: 24 items = 192 blocks -> again:
    # C = au(cd(960,000, 296), 256) = au(3244, 256) = 3328, now a short base: cd(40000, 3328) = 13 -> 16, and 40000 * 128 =
    # 5,120,000 >= 8 * 3328 * 181 = 4,818,944 keeps 16: chunks of au(2500, 256) = 2560, 16 each
    pl = P.plan([40000] * 3, 8, P.PlanParams())
    assert pl.chunk_target == 3328 and pl.num_splits == [16] * 3 and pl.chunk_len == [2560] * 3
    # a short base is never cut finer: 2 sequences of 3000 on 148 slots (C = 512, 8 heads): 2 * 8 * 2 * ... stays
    pl = P.plan([3000, 3000], 8, P.PlanParams())
    assert pl.chunk_target == 512 and pl == P.plan([3000, 3000], 8, P.PlanParams(refine=0))
    # one and a half waves or more stand: 28 x 20000 -> C = au(cd(4,480,000, 148), 256) = 30464, one chunk each:
    # 28 * 8 = 224 blocks, 448 >= 444
    pl = P.plan([20000] * 28, 8, P.PlanParams())
    assert pl.chunk_target == 30464 and pl.num_splits == [1] * 28
    # 27 x 20000 -> 216 blocks, 432 < 444: cut
    pl = P.plan([20000] * 27, 8, P.PlanParams())
    assert pl.chunk_target == au_ref(cd_ref(27 * 20000 * 8, 296), 256) and pl.num_splits == [2] * 27


def cd_ref(a, b):
    return (a + b - 1) // b


def au_ref(a, b):
    return cd_ref(a, b) * b
