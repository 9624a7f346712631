"""CPU oracle for the KV migration copies.  TEST INFRASTRUCTURE (only tests, the smoke check and the
benchmark's CPU baseline leg may import it).

The paper migrates a paused request between rollout buckets by offloading its KV cache, resharding it
along the attention-head dimension to the target tensor-parallel degree (a source partition is split
into TP_tgt / TP_src shards, or TP_src / TP_tgt partitions are concatenated) and reloading it
(Section 5.3).  These are pure rearrangements; the functions below are their definitions with explicit
indexing, on bf16 bit patterns (uint16), HND pools [page, head, slot, d].
"""
from __future__ import annotations

import numpy as np


def gather(pages: np.ndarray, block_table: np.ndarray, seq_lens, head_begin: int, head_count: int) -> np.ndarray:
    """Dense shard [total_tokens, head_count, d]: sequences one after the other, tokens in order."""
    rows = []
    P = pages.shape[2]
    for b, L in enumerate(seq_lens):
        for t in range(int(L)):
            rows.append(pages[block_table[b, t // P], head_begin:head_begin + head_count, t % P, :])
    if not rows:
        return np.zeros((0, head_count, pages.shape[3]), dtype=pages.dtype)
    return np.stack(rows)


def scatter(dense: np.ndarray, pages: np.ndarray, block_table: np.ndarray, seq_lens, head_begin: int) -> None:
    """Inverse of gather, in place: dense rows go to the pages `block_table` names, at head offset head_begin."""
    n = dense.shape[1]
    P = pages.shape[2]
    row = 0
    for b, L in enumerate(seq_lens):
        for t in range(int(L)):
            pages[block_table[b, t // P], head_begin:head_begin + n, t % P, :] = dense[row]
            row += 1


def split_heads(dense: np.ndarray, parts: int):
    """TP_tgt > TP_src: one partition becomes `parts` shards of consecutive heads."""
    n = dense.shape[1]
    assert n % parts == 0
    return [dense[:, i * (n // parts):(i + 1) * (n // parts), :] for i in range(parts)]


def concat_heads(shards) -> np.ndarray:
    """TP_tgt < TP_src: contiguous partitions are concatenated along the head axis."""
    return np.concatenate(list(shards), axis=1)
