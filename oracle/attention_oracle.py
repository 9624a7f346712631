"""CPU oracle for single-token GQA attention over a paged KV cache.  TEST INFRASTRUCTURE.

This file is the yardstick the CUDA library is measured against.  It is slow on
purpose, shares no code with the library or its Python binding, and must never be
imported by the product path: only tests, the smoke check and the benchmark's CPU
baseline leg may call it.

What it computes.  The paper's rollout stage is autoregressive decoding: every step
reads the whole KV cache of every running trajectory once per layer, which is why the
stage is bandwidth-bound and linear in sequence length (Section 1; Section 2.2,
"stage asymmetry").  The KV cache is organised by attention head (Section 5.3, step 2
of the migration).  The paper prints no formula for the attention itself; the
operation is the textbook one, written out here as its definition.  For sequence b
with L cached tokens (the current one included), query head h and KV head
g = h // G (G = query heads per KV head, contiguous groups):

    K_b[t] = k_pages[block_table[b, t // p], slot t % p, head g]      t = 0 .. L-1
    s_t    = (q[b, h] . K_b[t]) * sm_scale          sm_scale = 1 / sqrt(head_dim)
    out[b, h] = sum_t softmax(s)_t * V_b[t]
    lse[b, h] = ln sum_t exp(s_t)

All arithmetic is float64 on the exactly converted bf16 inputs.  An empty sequence
(L = 0) has out = 0 and lse = -inf.  Splitting the KV range, online softmax and the
log-sum-exp merge used by the library are re-associations of this sum, so none of them
appears here except ``merge_partials``, which states the merge identity itself so that
it can be checked against the direct formula.

Parity pins (tests/test_oracle_pins.py): length-1 returns v_0; identical V rows return
that row; zero query gives the mean of V (closed-form rational with integer V); a
dominant one-hot key returns exactly its value row; page placement does not matter;
shifting every key by u shifts every score by q.u*scale and nothing else; a dense,
loop-only brute force agrees on tiny inputs; chunked evaluation plus merge equals the
direct formula; an analytic two-token case.  The several-query-token form is pinned by
its reduction to the single-token function row by row, by the loop-only brute force, by
one-hot keys planted on either side of each query token's causal limit, and by the
zero-query running mean in closed form.  The E4M3 decoder is pinned by the format's
landmark values and by a library conversion of all 256 codes; the E4M3-cache form by its
equality with the bf16 definition on the decoded values (every E4M3 value is a bf16 value)
and by the scale identities.
"""
from __future__ import annotations

import math

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exact (bf16 is the top half of a float32)."""
    u32 = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


def gather_sequence(pages: np.ndarray, block_row: np.ndarray, length: int, layout: str = "HND") -> np.ndarray:
    """Rows of one sequence, in token order: float64[Hkv, length, d].

    pages: uint16 bf16 bits, "HND" = [num_pages, Hkv, page_size, d], "NHD" = [num_pages, page_size, Hkv, d].
    """
    if layout == "HND":
        page_size = pages.shape[2]
    elif layout == "NHD":
        page_size = pages.shape[1]
    else:
        raise ValueError(layout)
    n_pages = (length + page_size - 1) // page_size
    ids = np.asarray(block_row[:n_pages], dtype=np.int64)
    if np.any(ids < 0) or np.any(ids >= pages.shape[0]):
        raise IndexError("block table entry outside the pool")
    got = pages[ids]  # [n_pages, ...]
    if layout == "NHD":
        got = got.transpose(0, 2, 1, 3)  # -> [n_pages, Hkv, page, d]
    hkv, d = got.shape[1], got.shape[3]
    rows = got.transpose(1, 0, 2, 3).reshape(hkv, n_pages * page_size, d)[:, :length]
    return bf16_bits_to_f64(rows)


def paged_decode_attention(q, k_pages, v_pages, block_table, seq_lens, layout: str = "HND",
                           sm_scale: float | None = None, sequences=None):
    """The definition above for every sequence (or those listed in ``sequences``).

    q: uint16[B, Hq, d] bf16 bits.  Returns (out float64[B, Hq, d], lse float64[B, Hq]);
    rows of sequences that were not asked for are NaN.
    """
    q = np.asarray(q)
    B, Hq, d = q.shape
    Hkv = k_pages.shape[1] if layout == "HND" else k_pages.shape[2]
    assert Hq % Hkv == 0
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(d) if sm_scale is None else float(sm_scale)
    out = np.full((B, Hq, d), np.nan, dtype=np.float64)
    lse = np.full((B, Hq), np.nan, dtype=np.float64)
    todo = range(B) if sequences is None else sequences
    for b in todo:
        L = int(seq_lens[b])
        if L == 0:
            out[b] = 0.0
            lse[b] = -np.inf
            continue
        K = gather_sequence(k_pages, block_table[b], L, layout)      # [Hkv, L, d]
        V = gather_sequence(v_pages, block_table[b], L, layout)
        qb = bf16_bits_to_f64(q[b]).reshape(Hkv, G, d)               # head h = g * G + i
        s = np.matmul(qb, K.transpose(0, 2, 1)) * scale              # [Hkv, G, L]
        m = s.max(axis=2, keepdims=True)
        e = np.exp(s - m)
        z = e.sum(axis=2, keepdims=True)
        out[b] = np.matmul(e / z, V).reshape(Hq, d)
        lse[b] = (m + np.log(z)).reshape(Hq)
    return out, lse


def paged_multi_token_attention(q, k_pages, v_pages, block_table, seq_lens, layout: str = "HND",
                                sm_scale: float | None = None):
    """Several query tokens per sequence: the last Tq tokens of every sequence are new in this step
    (a tool return or a few drafted tokens appended at once; Section 2.2 describes how tool returns
    extend a trajectory mid-rollout).  Their K and V rows are already in the cache and seq_lens
    counts them.  Query token i (i = 0 .. Tq-1) sits at position L - Tq + i and, being causal,
    attends to cached tokens 0 .. L - Tq + i:

        n_i = L - Tq + 1 + i
        out[b, i, h] = sum_{t < n_i} softmax(s_0 .. s_{n_i - 1})_t * V_b[t],   s_t = (q[b, i, h] . K_b[t]) * sm_scale

    A query token with n_i <= 0 (a sequence shorter than Tq) has out = 0, lse = -inf.
    q: uint16[B, Tq, Hq, d].  Returns (out float64[B, Tq, Hq, d], lse float64[B, Tq, Hq]).
    Tq = 1 is the single-token definition above.
    """
    q = np.asarray(q)
    B, Tq, Hq, d = q.shape
    Hkv = k_pages.shape[1] if layout == "HND" else k_pages.shape[2]
    assert Hq % Hkv == 0
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(d) if sm_scale is None else float(sm_scale)
    out = np.zeros((B, Tq, Hq, d), dtype=np.float64)
    lse = np.full((B, Tq, Hq), -np.inf, dtype=np.float64)
    for b in range(B):
        L = int(seq_lens[b])
        if L == 0:
            continue
        K = gather_sequence(k_pages, block_table[b], L, layout)      # [Hkv, L, d]
        V = gather_sequence(v_pages, block_table[b], L, layout)
        for i in range(Tq):
            n = L - Tq + 1 + i
            if n <= 0:
                continue
            qi = bf16_bits_to_f64(q[b, i]).reshape(Hkv, G, d)
            s = np.matmul(qi, K[:, :n].transpose(0, 2, 1)) * scale   # [Hkv, G, n]
            m = s.max(axis=2, keepdims=True)
            e = np.exp(s - m)
            z = e.sum(axis=2, keepdims=True)
            out[b, i] = np.matmul(e / z, V[:, :n]).reshape(Hq, d)
            lse[b, i] = (m + np.log(z)).reshape(Hq)
    return out, lse


def e4m3_to_f64(codes: np.ndarray) -> np.ndarray:
    """8-bit floating point, 1 sign / 4 exponent / 3 mantissa bits, bias 7, no infinities ("E4M3", the
    common KV-cache storage format) -> float64, exact.  Written from the format's definition:
    exponent field 0 is subnormal (m / 8 * 2^-6), field e >= 1 is (1 + m / 8) * 2^(e - 7); the one
    all-ones pattern per sign (e = 15, m = 7) is NaN; the largest finite value is 448."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 0x7).astype(np.float64)
    mag = np.where(e == 0, m / 8.0 * 2.0 ** -6, (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64)))
    mag = np.where((e == 15) & (m == 7), np.nan, mag)
    return sign * mag


def paged_decode_attention_fp8(q, k_pages8, v_pages8, block_table, seq_lens, k_scale: float = 1.0,
                               v_scale: float = 1.0, sm_scale: float | None = None):
    """Single-token decode over a KV cache stored as E4M3 codes with one scale per tensor: the cached
    key of token t is k_scale * e4m3(k code), the value v_scale * e4m3(v code); everything else is the
    definition at the top of this file, in float64.  Pools: uint8 [num_pages, Hkv, page_size, d] (HND).
    q: uint16 bf16 bits [B, Hq, d].  Returns (out float64[B, Hq, d], lse float64[B, Hq])."""
    q = np.asarray(q)
    B, Hq, d = q.shape
    Hkv, page_size = k_pages8.shape[1], k_pages8.shape[2]
    assert Hq % Hkv == 0
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(d) if sm_scale is None else float(sm_scale)
    out = np.zeros((B, Hq, d), dtype=np.float64)
    lse = np.full((B, Hq), -np.inf, dtype=np.float64)
    for b in range(B):
        L = int(seq_lens[b])
        if L == 0:
            continue
        n_pages = (L + page_size - 1) // page_size
        ids = np.asarray(block_table[b, :n_pages], dtype=np.int64)
        if np.any(ids < 0) or np.any(ids >= k_pages8.shape[0]):
            raise IndexError("block table entry outside the pool")
        K = e4m3_to_f64(k_pages8[ids].transpose(1, 0, 2, 3).reshape(Hkv, n_pages * page_size, d)[:, :L]) * float(k_scale)
        V = e4m3_to_f64(v_pages8[ids].transpose(1, 0, 2, 3).reshape(Hkv, n_pages * page_size, d)[:, :L]) * float(v_scale)
        qb = bf16_bits_to_f64(q[b]).reshape(Hkv, G, d)
        s = np.matmul(qb, K.transpose(0, 2, 1)) * scale
        m = s.max(axis=2, keepdims=True)
        e = np.exp(s - m)
        z = e.sum(axis=2, keepdims=True)
        out[b] = np.matmul(e / z, V).reshape(Hq, d)
        lse[b] = (m + np.log(z)).reshape(Hq)
    return out, lse


def dense_attention_loops(q_row, K, V, scale: float):
    """Loop-only softmax(q K^T * scale) V for ONE head on dense float64 rows: the brute
    force the paged oracle is checked against.  q_row[d], K[L, d], V[L, d] (lists or arrays)."""
    L = len(K)
    d = len(q_row)
    s = []
    for t in range(L):
        acc = 0.0
        for j in range(d):
            acc += float(q_row[j]) * float(K[t][j])
        s.append(acc * scale)
    m = max(s)
    e = [math.exp(x - m) for x in s]
    z = math.fsum(e)
    o = [math.fsum(e[t] * float(V[t][j]) for t in range(L)) / z for j in range(d)]
    return o, m + math.log(z)


def merge_partials(outs, lses):
    """Log-sum-exp merge of per-chunk results of one head (step C of the path):
    M = max_i lse_i, w_i = exp(lse_i - M), out = sum_i w_i out_i / sum_i w_i,
    lse = M + ln sum_i w_i.  outs: float64[n, d], lses: float64[n]."""
    outs = np.asarray(outs, dtype=np.float64)
    lses = np.asarray(lses, dtype=np.float64)
    M = lses.max()
    if not np.isfinite(M):
        return np.zeros(outs.shape[1]), -np.inf
    w = np.exp(lses - M)
    return (w[:, None] * outs).sum(axis=0) / w.sum(), M + math.log(w.sum())


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest bf16 value (ties to even), returned as float64.  Used by tests that
    compare against the library's bf16 output bit for bit where the exact result is a bf16 value."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32)
    r = ((u + (((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))) >> np.uint32(16)) << np.uint32(16)
    return r.view(np.float32).astype(np.float64)
