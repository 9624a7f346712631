"""Reference work planner (plain Python integers).  TEST INFRASTRUCTURE.

Independent restatement of the planning rule the CUDA library implements in C++; the
two share no code and are compared bit for bit.  Only tests, the smoke check and the
benchmark's CPU baseline leg may import this file.

Where the rule comes from.  The paper removes rollout stragglers by splitting the
rollout cluster into buckets ordered by capacity, each with its own parallel degree
taken from {1, 2, 4, 8}, and by sending longer requests to higher degrees (Section 2.3
"Rollout Optimizations"; Section 4.3: degree set, requests sorted by length, contiguous
segments, objective = smallest maximum completion time; Section 5: buckets ordered by
capacity, histogram bins aligned with bucket thresholds).  On one GPU the "workers" are
the resident thread blocks and the "degree" of a sequence is the number of blocks that
share its KV range, so:

  * bucket k holds the sequences whose length lies in (C * 2^(k-1), C * 2^k]; bucket 0
    is (0, C]; the degree of bucket k is 2^k, capped at S_max;
  * when C is short (C < 4096 tokens, where the fixed cost of a work item shows), the
    bucket limits move up to the geometric means of those limits: a sequence of bucket
    k >= 1 with L * 128 < 2^(k-1) * C * 181 (181 / 128 ~ sqrt 2) takes degree 2^(k-1),
    the power of two nearer to L / C in ratio;
  * C, the base length, is recomputed for every batch from the total work so that the
    launch has about `items_per_slot` work items per resident block;
  * items are issued longest first (the classic greedy rule for the min-max objective);
  * coarse plans are cut finer: when the base is long (C >= 4096 tokens) and the plan has fewer than one and a
    half waves of blocks (2 * Hkv * sum n_b < 3 * W), the base is recomputed for twice as many slots and every
    sequence is bucketed again.  This is the tail end of a rollout, when only a few long stragglers are still
    decoding (Section 2.2): with so few blocks the second wave leaves most SMs idle and the blocks that run cannot
    pull the memory bandwidth alone (measured on a B200: 12 sequences of 20,000 tokens 169 -> 147 us, 26 sequences
    of 16K-32K tokens 420 -> 389 us, while batches with at least 1.5 waves lose 1-3 % when cut finer).

The paper states no single-GPU rule; this is the reading this library takes.

All arithmetic is integer.  cd(a, b) = ceil(a / b); au(a, b) = cd(a, b) * b;
p2(x) = least power of two >= x.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass(frozen=True)
class PlanParams:
    n_sm: int = 148
    ctas_per_sm: int = 1
    items_per_slot: int = 1
    chunk_align: int = 256      # A: chunk lengths are multiples of this many tokens
    min_chunk: int = 512        # C_min
    max_splits: int = 64        # S_max
    small_base: int = 4096      # base lengths below this take the nearer power of two (0 = never: the plain rule)
    refine: int = 1             # 1: plans of fewer than 1.5 waves of long blocks are cut twice as fine (0 = never)


REFINE_MIN_BASE = 4096   # bases shorter than this are never cut finer: there the fixed cost of a block dominates


def cd(a: int, b: int) -> int:
    return -(-a // b)


def au(a: int, b: int) -> int:
    return cd(a, b) * b


def p2(x: int) -> int:
    r = 1
    while r < x:
        r *= 2
    return r


@dataclass
class Plan:
    chunk_target: int            # C
    bucket: list                 # per sequence: log2(split degree), -1 for an empty sequence
    num_splits: list             # n_b: non-empty chunks of sequence b
    chunk_len: list              # chunk_b
    item_offset: list            # exclusive prefix sum of n_b (batch order)
    items: list                  # sorted work list of (b, j, kv_begin, kv_end)
    combine: list                # sequences with n_b > 1, batch order
    empty: list                  # sequences with L_b == 0, batch order


def plan(seq_lens, num_kv_heads: int, params: PlanParams = PlanParams()) -> Plan:
    lens = [int(x) for x in seq_lens]
    if any(L < 0 for L in lens):
        raise ValueError("negative sequence length")
    W = params.n_sm * params.ctas_per_sm
    T = sum(lens)
    A = params.chunk_align
    C = max(params.min_chunk, au(cd(num_kv_heads * T, W * params.items_per_slot), A))

    def per_sequence(C):
        bucket, nsplit, chunk = [], [], []
        for L in lens:
            if L == 0:
                bucket.append(-1); nsplit.append(0); chunk.append(0)
                continue
            s = p2(cd(L, C))
            if C < params.small_base and s > 1 and L * 128 < (s // 2) * C * 181:
                s //= 2
            s = min(s, params.max_splits)
            c = au(cd(L, s), A)
            bucket.append(s.bit_length() - 1)
            chunk.append(c)
            nsplit.append(cd(L, c))
        return bucket, nsplit, chunk

    bucket, nsplit, chunk = per_sequence(C)
    # a coarse plan of long blocks (fewer than one and a half waves) is made again for twice as many slots
    if params.refine and C >= REFINE_MIN_BASE and 2 * num_kv_heads * sum(nsplit) < 3 * W:
        C = max(params.min_chunk, au(cd(num_kv_heads * T, 2 * W * params.items_per_slot), A))
        bucket, nsplit, chunk = per_sequence(C)
    offs, run = [], 0
    for n in nsplit:
        offs.append(run)
        run += n
    items = []
    for b, L in enumerate(lens):
        for j in range(nsplit[b]):
            items.append((b, j, j * chunk[b], min(L, (j + 1) * chunk[b])))
    items.sort(key=lambda it: (-(it[3] - it[2]), it[0], it[1]))
    return Plan(C, bucket, nsplit, chunk, offs, items,
                [b for b, n in enumerate(nsplit) if n > 1],
                [b for b, L in enumerate(lens) if L == 0])
