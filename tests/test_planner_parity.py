"""The library's C++ planner against the independent Python reference planner: bit-exact on the
five workloads, on random length vectors and on edge cases.  Pure host code, no GPU."""
import numpy as np
import pytest

from oracle import planner_ref as P
from paper_2606_03077_b200 import workloads as W


def both(lib, lens, hkv, prm: P.PlanParams):
    ref = P.plan(lens, hkv, prm)
    got = lib.libra_plan_host(lens, hkv, lib.PlanParams(prm.n_sm, prm.ctas_per_sm, prm.items_per_slot,
                                                        prm.chunk_align, prm.min_chunk, prm.max_splits,
                                                        1 if prm.refine else -1))
    assert got["chunk_target"] == ref.chunk_target
    assert list(got["bucket"]) == ref.bucket
    assert list(got["num_splits"]) == ref.num_splits
    assert list(got["chunk_len"]) == ref.chunk_len
    assert list(got["item_offset"]) == ref.item_offset
    assert [tuple(r) for r in got["items"]] == ref.items
    assert list(got["combine"]) == ref.combine
    assert list(got["empty"]) == ref.empty
    return ref


@pytest.mark.parametrize("name", W.WORKLOAD_ORDER)
def test_workloads_bit_exact(lib, name):
    w = W.WORKLOADS[name]
    for step in range(w.steps):
        lay, _ = W.make_layout(name, step)
        both(lib, lay.seq_lens, w.num_kv_heads, P.PlanParams())


def test_random_vectors_bit_exact(lib):
    rng = np.random.default_rng(5)
    for i in range(300):
        B = int(rng.integers(1, 257))
        lens = np.clip(np.floor(rng.choice([16, 300, 2000, 12000]) * np.exp(rng.normal(size=B) * rng.uniform(0.2, 1.5))),
                       0, 40960).astype(np.int32)
        prm = P.PlanParams(n_sm=int(rng.choice([1, 2, 74, 148])), ctas_per_sm=int(rng.integers(1, 5)),
                           items_per_slot=int(rng.integers(1, 9)), chunk_align=int(rng.choice([16, 64, 256, 512])),
                           min_chunk=int(rng.choice([16, 512, 2048])), max_splits=int(rng.choice([1, 2, 8, 64])))
        both(lib, lens, int(rng.choice([1, 2, 4, 8])), prm)


def test_few_long_sequences_bit_exact(lib):
    """Small batches of long sequences on many slots: plans of fewer than one and a half waves, which are made again
    for twice as many slots."""
    import dataclasses
    rng = np.random.default_rng(6)
    refined = 0
    for i in range(400):
        B = int(rng.integers(1, 40))
        base = int(rng.choice([3000, 12000, 20000, 30000]))
        if i % 3 == 0:
            lens = np.full(B, base, dtype=np.int32)
        else:
            lens = np.clip(np.floor(base * np.exp(rng.normal(size=B) * rng.uniform(0.05, 0.8))), 0, 40960).astype(np.int32)
        hkv = int(rng.choice([1, 2, 4, 8]))
        for rf in (1, 0):
            prm = P.PlanParams(n_sm=int(rng.choice([16, 74, 148, 296])), ctas_per_sm=int(rng.integers(1, 3)),
                               items_per_slot=int(rng.integers(1, 3)), chunk_align=int(rng.choice([16, 256])),
                               min_chunk=int(rng.choice([16, 512])), max_splits=int(rng.choice([2, 8, 64])), refine=rf)
            ref = both(lib, lens, hkv, prm)
            refined += ref != P.plan(lens, hkv, dataclasses.replace(prm, refine=0))
    assert refined > 30   # the cases did exercise the rule


def test_edge_cases(lib):
    prm = P.PlanParams()
    both(lib, np.zeros(0, np.int32), 8, prm)                       # empty batch
    both(lib, np.zeros(5, np.int32), 8, prm)                       # only empty sequences
    both(lib, np.array([1], np.int32), 1, prm)
    both(lib, np.array([40960] * 256, np.int32), 8, prm)           # everything at the paper's length cap
    both(lib, np.array([16, 17, 255, 256, 257, 511, 512, 513], np.int32), 8, prm)
    both(lib, np.array([2 ** 20], np.int32), 8, prm)               # degree capped at max_splits
    ties = both(lib, np.array([1024] * 7 + [2048] * 3, np.int32), 2, P.PlanParams(n_sm=4))
    assert len({(b, j) for b, j, _, _ in ties.items}) == len(ties.items)


def test_bad_arguments(lib):
    ok = lib.PlanParams(148, 2, 4, 256, 512, 64)
    with pytest.raises(lib.LibraError) as e:
        lib.libra_plan_host([5, -1], 8, ok)
    assert e.value.status == lib.INVALID_ARGUMENT
    for bad in (lib.PlanParams(0, 2, 4, 256, 512, 64), lib.PlanParams(148, 2, 4, 100, 512, 64),
                lib.PlanParams(148, 2, 4, 256, 512, 48), lib.PlanParams(148, 2, 4, 256, 512, 128)):
        with pytest.raises(lib.LibraError) as e:
            lib.libra_plan_host([5], 8, bad)
        assert e.value.status == lib.INVALID_ARGUMENT
    with pytest.raises(lib.LibraError) as e:
        lib.libra_plan_host([100000], 8, ok, items_capacity=2)
    assert e.value.status == lib.WORKSPACE_TOO_SMALL


def test_item_bound_holds(lib):
    # sum n_b <= 2*ceil(W*ips / Hkv) + B, the bound the workspace is sized by; a refined plan is a plan for twice the slots
    rng = np.random.default_rng(6)
    for i in range(300):
        B = int(rng.integers(1, 257 if i % 2 else 12)); hkv = int(rng.choice([1, 2, 8]))
        lens = rng.integers(0, 40961, B).astype(np.int32)
        for refine in (0, 1):
            prm = P.PlanParams(n_sm=int(rng.choice([4, 148])), items_per_slot=int(rng.integers(1, 6)), refine=refine)
            pl = P.plan(lens, hkv, prm)
            W_ = prm.n_sm * prm.ctas_per_sm * prm.items_per_slot
            plain = 2 * (-(-W_ // hkv)) + B
            few = min(B, (3 * prm.n_sm * prm.ctas_per_sm) // (2 * hkv))
            assert len(pl.items) <= (max(plain, 2 * (-(-2 * W_ // hkv)) + few) if refine else plain)
