"""CPU oracle for the data plane of the ring all-reduce.  TEST INFRASTRUCTURE (only tests, the smoke check and the
benchmark's CPU baseline leg may import it).

The paper exchanges gradients between replicas with a ring algorithm, ReduceScatter followed by AllGather, whose
GPU side only copies and reduces chunks while the CPU owns membership and transport (Section 6, "Decoupled
communication domains"; appendix "Decoupled Communication Domain").  The paper prints no formula; the ring
algorithm is the textbook one, written out here step by step so that the order of the additions is fixed:

  R ranks, each with a vector x_r cut into R chunks (chunk c = elements [bounds[c], bounds[c+1])).
  ReduceScatter, steps s = 0 .. R-2: rank r sends its current chunk (r - s) mod R to rank r+1, which adds it to its
      own copy of that chunk:  x_{r+1}[c] = x_{r+1}[c] + received.
      After R-1 steps rank r holds the complete sum of chunk (r + 1) mod R.
  AllGather, steps s = 0 .. R-2: rank r sends chunk (r + 1 - s) mod R to rank r+1, which overwrites its copy.

Additions are done in the element type of the exchange (float32, or bfloat16 with the sum formed in float32 and
rounded to nearest even after every step), so the result is defined bit for bit; every rank ends with the same
vector.  Pins (tests/test_oracle_ring.py): the float64 sum within rounding; exact sums of small integers; R = 1 is
the identity, R = 2 is x_0 + x_1; every rank ends identical; the per-chunk order of additions stated above.
"""
from __future__ import annotations

import numpy as np


def chunk_bounds(n: int, ranks: int, granule: int = 1) -> list[int]:
    """Chunk c covers [bounds[c], bounds[c+1]): equal parts, the first ones one unit longer.  The unit is `granule`
    elements (1 by default; a transport that moves whole 16-byte vectors cuts at multiples of 16 bytes: granule 4
    for float32, 8 for bfloat16); n must be a multiple of it.  The paper does not say where a vector is cut."""
    if n % granule:
        raise ValueError("vector length is not a multiple of the granule")
    base, extra = divmod(n // granule, ranks)
    bounds = [0]
    for c in range(ranks):
        bounds.append(bounds[-1] + (base + (1 if c < extra else 0)) * granule)
    return bounds


def _bf16_round(x32: np.ndarray) -> np.ndarray:
    """float32 -> nearest bfloat16 (ties to even), returned as float32."""
    u = x32.astype(np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def add_step(own: np.ndarray, received: np.ndarray, dtype: str) -> np.ndarray:
    """One reduction step in the exchange's element type."""
    if dtype == "f32":
        return (own.astype(np.float32) + received.astype(np.float32)).astype(np.float32)
    if dtype == "bf16":     # values held as float32 that are exact bf16 numbers
        return _bf16_round(own.astype(np.float32) + received.astype(np.float32))
    raise ValueError(dtype)


def ring_all_reduce(xs, dtype: str = "f32", granule: int = 1):
    """xs: list of R equal-length float32 arrays (for "bf16": exact bf16 values).  Returns the R result vectors."""
    R = len(xs)
    n = len(xs[0])
    bounds = chunk_bounds(n, R, granule)
    bufs = [np.array(x, dtype=np.float32, copy=True) for x in xs]
    sl = lambda c: slice(bounds[c % R], bounds[c % R + 1])
    for s in range(R - 1):                       # ReduceScatter
        sent = [bufs[r][sl(r - s)].copy() for r in range(R)]        # all ranks send at once
        for r in range(R):
            dst = (r + 1) % R
            bufs[dst][sl(r - s)] = add_step(bufs[dst][sl(r - s)], sent[r], dtype)
    for s in range(R - 1):                       # AllGather
        sent = [bufs[r][sl(r + 1 - s)].copy() for r in range(R)]
        for r in range(R):
            bufs[(r + 1) % R][sl(r + 1 - s)] = sent[r]
    return bufs
