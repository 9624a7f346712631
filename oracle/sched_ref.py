"""Reference implementations of the paper's rollout-side schedulers.  TEST INFRASTRUCTURE.

* ``rollout_partition_brute_force``: the problem RolloutDP solves (Section 4.3), by exhaustive search:
  every way to split the GPUs into instances with degrees from T, every way to cut the length-sorted
  requests into that many contiguous (possibly empty) segments; the makespan is the largest instance
  cost.  Exponential: tiny inputs only.  The DP must find the same optimum.
* ``PrefixTree``: the causality-aware prefix tree and the routing rule of Section 5, with dictionaries.
"""
from __future__ import annotations

import itertools
import math


def segment_cost(coef, lens_sorted, first, count):
    """Polynomial instance cost on sorted requests [first, first + count): a*sum L + b*sum L^2 + c*count + d."""
    if count == 0:
        return 0.0
    seg = lens_sorted[first:first + count]
    a, b, c, d = coef
    return a * sum(seg) + b * sum(x * x for x in seg) + c * count + d


def rollout_partition_brute_force(n_gpus, lengths, tp_set, cost_coef):
    lens = sorted(int(x) for x in lengths)
    L = len(lens)
    best = math.inf

    def degree_sequences(g):
        if g == 0:
            yield []
            return
        for t, tp in enumerate(tp_set):
            if tp <= g:
                for rest in degree_sequences(g - tp):
                    yield [t] + rest

    for seq in degree_sequences(n_gpus):
        m = len(seq)
        if m == 0:
            if L == 0:
                best = min(best, 0.0)
            continue
        # cut points 0 = c_0 <= c_1 <= ... <= c_m = L
        for cuts in itertools.combinations_with_replacement(range(L + 1), m - 1):
            bounds = [0] + list(cuts) + [L]
            cost = max(segment_cost(cost_coef[seq[k]], lens, bounds[k], bounds[k + 1] - bounds[k]) for k in range(m))
            best = min(best, cost)
    return best


class PrefixTree:
    def __init__(self, bin_upper):
        self.bin_upper = list(bin_upper)
        self.hist = {}  # key (prompt, (s1, ..., sk)) -> counts per bin

    def _bin(self, length):
        for k, u in enumerate(self.bin_upper):
            if length <= u:
                return k
        return len(self.bin_upper)

    def insert(self, prompt, states, residuals):
        for k in range(len(states) + 1):
            key = (prompt, tuple(states[:k]))
            h = self.hist.setdefault(key, [0] * (len(self.bin_upper) + 1))
            h[self._bin(residuals[k])] += 1

    def lookup(self, prompt, states):
        if (prompt, ()) not in self.hist:
            return [0.0] * (len(self.bin_upper) + 1), -1, 0
        depth = 0
        while depth < len(states) and (prompt, tuple(states[:depth + 1])) in self.hist:
            depth += 1
        h = self.hist[(prompt, tuple(states[:depth]))]
        n = sum(h)
        return [x / n for x in h], depth, n

    def route(self, prompt, states, decode_cost, migration_cost):
        p, _, _ = self.lookup(prompt, states)
        costs = [migration_cost[b] + sum(p[k] * decode_cost[b][k] for k in range(len(p))) for b in range(len(migration_cost))]
        best = min(range(len(costs)), key=lambda b: (costs[b], b))
        return best, costs[best]
