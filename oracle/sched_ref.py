"""Reference implementations of the paper's rollout-side schedulers.  TEST INFRASTRUCTURE.

* ``rollout_partition_brute_force``: the problem RolloutDP solves (Section 4.3), by exhaustive search:
  every way to split the GPUs into instances with degrees from T, every way to cut the length-sorted
  requests into that many contiguous (possibly empty) segments; the makespan is the largest instance
  cost.  Exponential: tiny inputs only.  The DP must find the same optimum.
* ``rollout_dp_scan``: the recurrence itself, every term tried; the library's evaluation (bisection, or forward
  relaxation) must give the same makespan and the same partition, ties included.
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


def rollout_dp_scan(n_gpus, lengths, tp_set, cost_coef):
    """The recurrence of Section 4.3 evaluated term by term (every degree, every x), in float64:

        dp[g][i] = min over t with tp_t <= g, 0 <= x <= i of max(dp[g - tp_t][i - x], Cost(t, i - x + 1, i))

    dp[0][0] = 0, everything else starts at +inf ("exactly g GPUs serve the first i sorted requests"); Cost is the
    polynomial a * sum L + b * sum L^2 + c * count + d on the segment's prefix sums, 0 for an empty segment.  Ties go to
    the earlier degree, then to the smaller x.  Returns (makespan, [(tp, first_sorted_index, count), ...]) with the
    instances in sorted-request order, or (inf, []) when no partition uses exactly n_gpus GPUs.  Polynomial time, but
    slow: small and medium inputs only.  Pinned by the exhaustive search above."""
    import numpy as np
    lens = sorted(int(x) for x in lengths)
    L, G = len(lens), int(n_gpus)
    s1, s2 = [0.0], [0.0]
    for v in lens:
        s1.append(s1[-1] + float(v))
        s2.append(s2[-1] + float(v) * float(v))
    s1, s2 = np.array(s1), np.array(s2)
    dp = np.full((G + 1, L + 1), np.inf)
    arg = {}
    dp[0, 0] = 0.0
    for g in range(1, G + 1):
        for i in range(L + 1):
            best, bt, bx = math.inf, -1, -1
            xs = np.arange(i + 1)
            for t, tp in enumerate(tp_set):
                if tp > g:
                    continue
                a, b, c, d = (float(v) for v in cost_coef[t])
                seg = a * (s1[i] - s1[i - xs]) + b * (s2[i] - s2[i - xs]) + c * xs.astype(np.float64) + d
                seg[0] = 0.0                                   # the empty segment costs nothing
                cand = np.maximum(dp[g - tp, i - xs], seg)
                x = int(np.argmin(cand))                       # first minimum: the smallest x
                if cand[x] < best:
                    best, bt, bx = float(cand[x]), t, x
            dp[g, i] = best
            arg[(g, i)] = (bt, bx)
    if math.isinf(dp[G, L]):
        return math.inf, []
    inst, g, i = [], G, L
    while g > 0:
        t, x = arg[(g, i)]
        inst.append((int(tp_set[t]), i - x, x))
        g -= tp_set[t]
        i -= x
    return float(dp[G, L]), inst[::-1]


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
