"""The paper's rollout-side schedulers (host code in the library) against exhaustive search and a
dictionary implementation.  Pure CPU."""
import math

import numpy as np
import pytest

from oracle import sched_ref as R


def check_partition(lens, n_gpus, tp_set, coef, makespan, inst):
    ls = sorted(int(x) for x in lens)
    assert sum(tp for tp, _, _ in inst) == n_gpus                 # every GPU is used
    assert sum(c for _, _, c in inst) == len(ls)                  # every request is served once
    pos = 0
    worst = 0.0
    for tp, first, count in inst:                                 # contiguous segments of the sorted list, in order
        assert tp in tp_set and first == pos and count >= 0
        pos += count
        worst = max(worst, R.segment_cost(coef[list(tp_set).index(tp)], ls, first, count))
    assert worst == pytest.approx(makespan, rel=1e-12)


def test_hand_worked_case(lib):
    # 3 GPUs, degrees {1, 2}, cost = sum(L) / tp.  Requests 1, 2, 3, 10.
    # Best: TP-1 serves {1,2,3} (cost 6), TP-2 serves {10} (cost 5): makespan 6.
    coef = [[1.0, 0, 0, 0], [0.5, 0, 0, 0]]
    mk, inst = lib.libra_rollout_dp(3, [10, 1, 3, 2], [1, 2], coef)
    assert mk == 6.0
    assert inst == [(1, 0, 3), (2, 3, 1)]
    assert R.rollout_partition_brute_force(3, [10, 1, 3, 2], [1, 2], coef) == 6.0


def test_dp_matches_exhaustive_search(lib):
    rng = np.random.default_rng(0)
    for _ in range(120):
        n_gpus = int(rng.integers(1, 7))
        L = int(rng.integers(0, 7))
        lens = rng.integers(1, 60, L)
        tp_set = sorted(set(int(x) for x in rng.choice([1, 2, 4, 8], size=int(rng.integers(1, 4)))))
        coef = [[float(rng.uniform(0.1, 2)) / tp, float(rng.uniform(0, 0.05)) / tp, float(rng.uniform(0, 1)),
                 float(rng.uniform(0, 3))] for tp in tp_set]
        want = R.rollout_partition_brute_force(n_gpus, lens, tp_set, coef)
        mk, inst = lib.libra_rollout_dp(n_gpus, lens, tp_set, coef)
        if math.isinf(want):
            assert math.isinf(mk) and inst == []
        else:
            assert mk == pytest.approx(want, rel=1e-12)
            check_partition(lens, n_gpus, tp_set, coef, mk, inst)


def test_longer_requests_go_to_higher_degrees(lib):
    # the effect the paper describes (Section 2.3): small TP is cheaper per GPU on short requests (no
    # communication term), large TP wins on long ones (the quadratic term divides by tp)
    tp_set = [1, 2, 4, 8]
    coef = [[1.0 / tp + 0.2 * (tp - 1), 2e-4 / tp, 0.0, 0.0] for tp in tp_set]
    rng = np.random.default_rng(1)
    lens = np.concatenate([rng.integers(200, 2000, 40), rng.integers(16000, 32000, 8)])
    mk, inst = lib.libra_rollout_dp(16, lens, tp_set, coef)
    check_partition(lens, 16, tp_set, coef, mk, inst)
    used = [(tp, first, count) for tp, first, count in inst if count > 0]
    assert used[0][0] < used[-1][0]          # the segment of the longest requests runs at a higher degree
    assert mk < R.segment_cost(coef[0], sorted(int(x) for x in lens), 0, len(lens))   # better than one TP-1 instance


def test_dp_argument_errors(lib):
    with pytest.raises(lib.LibraError):
        lib.libra_rollout_dp(4, [5, 6], [0, 2], [[1, 0, 0, 0], [1, 0, 0, 0]])
    mk, inst = lib.libra_rollout_dp(3, [5, 6], [2], [[1, 0, 0, 0]])     # 3 GPUs cannot be split into TP-2 instances
    assert math.isinf(mk) and inst == []


def test_prefix_tree_against_dictionaries(lib):
    rng = np.random.default_rng(2)
    bins = [2048, 8192, 16384]
    t, ref = lib.Trie(bins), R.PrefixTree(bins)
    for _ in range(400):
        prompt = int(rng.integers(0, 5))
        n = int(rng.integers(0, 5))
        states = [int(x) for x in rng.integers(0, 4, n)]
        total = int(rng.integers(100, 40000))
        cuts = sorted(int(x) for x in rng.integers(0, total, n))
        residuals = [total] + [total - c for c in cuts]
        t.insert(prompt, states, residuals)
        ref.insert(prompt, states, residuals)
    decode_cost = [[1.0, 4.0, 16.0, 40.0], [1.6, 3.0, 9.0, 20.0], [2.5, 3.5, 6.0, 11.0]]
    for _ in range(300):
        prompt = int(rng.integers(0, 7))          # 5 and 6 were never inserted
        states = [int(x) for x in rng.integers(0, 5, int(rng.integers(0, 6)))]   # label 4 never seen: back-off
        h, d, n = t.lookup(prompt, states)
        hr, dr, nr = ref.lookup(prompt, states)
        assert d == dr and n == nr and np.allclose(h, hr, rtol=0, atol=1e-15)
        cur = int(rng.integers(0, 3))
        mig = [0.0 if b == cur else 1.5 + abs(b - cur) for b in range(3)]
        assert t.route(prompt, states, decode_cost, mig) == pytest.approx(ref.route(prompt, states, decode_cost, mig))
    t.close()


def test_prefix_tree_small_example(lib):
    t = lib.Trie([1000])
    t.insert(7, [1, 2], [5000, 3000, 500])     # after the second tool return only 500 tokens remained
    t.insert(7, [1, 3], [9000, 8000, 7000])
    h, d, n = t.lookup(7, [1])
    assert (list(h), d, n) == ([0.0, 1.0], 1, 2)
    h, d, n = t.lookup(7, [1, 2])
    assert (list(h), d, n) == ([1.0, 0.0], 2, 1)
    h, d, n = t.lookup(7, [1, 9, 2])            # unseen state 9: back off to the node of [1]
    assert (list(h), d, n) == ([0.0, 1.0], 1, 2)
    assert t.lookup(8, [])[1] == -1
    # short remainder expected: stay in the small bucket; long remainder: migrate although it costs
    cost = [[1.0, 10.0], [2.0, 4.0]]
    assert t.route(7, [1, 2], cost, [0.0, 1.0])[0] == 0
    assert t.route(7, [1, 3], cost, [0.0, 1.0])[0] == 1
    t.close()


def test_scan_reference_finds_the_exhaustive_optimum():
    """The term-by-term evaluation of the recurrence (the reference below) against exhaustive search."""
    rng = np.random.default_rng(17)
    for trial in range(40):
        n = int(rng.integers(0, 7)); g = int(rng.integers(1, 7))
        lens = rng.integers(1, 50, size=n)
        tp_set = sorted(set(int(x) for x in rng.choice([1, 2, 4], size=int(rng.integers(1, 4)))))
        coef = [[float(rng.integers(0, 4)), float(rng.integers(0, 3)) * 1e-2, float(rng.integers(0, 3)), float(rng.integers(0, 5))]
                for _ in tp_set]
        mk, inst = R.rollout_dp_scan(g, lens, tp_set, coef)
        want = R.rollout_partition_brute_force(g, lens, tp_set, coef)
        assert (math.isinf(mk) and math.isinf(want)) or abs(mk - want) <= 1e-9 * max(1.0, abs(want))
        if not math.isinf(mk):
            assert sum(tp for tp, _, _ in inst) == g and sum(c for _, _, c in inst) == n


def test_library_gives_the_recurrence_bit_for_bit(lib):
    """libra_rollout_dp (bisection on x where no coefficient is negative, forward relaxation otherwise) against the
    term-by-term evaluation of the recurrence: same makespan, same partition, ties included."""
    import time
    rng = np.random.default_rng(7)
    for trial in range(48):
        n = int(rng.integers(0, 90))
        g = int(rng.integers(1, 20))
        kind = trial % 4
        if kind == 0:
            lens = rng.integers(1, 40000, size=n)
        elif kind == 1:
            lens = rng.integers(1, 6, size=n)                    # many equal lengths: ties everywhere
        elif kind == 2:
            lens = np.full(n, 1000)
        else:
            lens = np.floor(1024 * np.exp(rng.standard_normal(n))).astype(np.int64) + 1
        tp_set = sorted(set(int(x) for x in rng.choice([1, 2, 4, 8], size=int(rng.integers(1, 5)))))
        coef = [[float(rng.integers(0, 4)) / (1 + t), float(rng.integers(0, 3)) * 1e-4 / (1 + t), float(rng.integers(0, 3)),
                 float(rng.integers(0, 5))] for t in range(len(tp_set))]
        if trial % 6 == 5:
            coef[0][2] = -0.5                                    # a negative coefficient: no bisection
        got = lib.libra_rollout_dp(g, lens, tp_set, coef)
        want = R.rollout_dp_scan(g, lens, tp_set, coef)
        assert got == want or (math.isinf(got[0]) and math.isinf(want[0])), (trial, got, want)
    rng = np.random.default_rng(8)
    # and it is what makes the planner cheap: 128 GPUs x 4096 requests
    lens = np.floor(2048 * np.exp(rng.standard_normal(4096))).astype(np.int64) + 1
    coef = [[1.0 / tp, 2e-5 / tp, 5.0, 100.0 * tp] for tp in (1, 2, 4, 8)]
    t0 = time.perf_counter()
    mk, inst = lib.libra_rollout_dp(128, lens, [1, 2, 4, 8], coef)
    dt = time.perf_counter() - t0
    assert math.isfinite(mk) and sum(c for _, _, c in inst) == 4096 and sum(tp for tp, _, _ in inst) == 128
    assert dt < 5.0
