"""Seeded synthetic inputs for paged GQA decode attention.

This module only draws random numbers and lays them out in pages.  It holds none
of the method's arithmetic (no softmax, no planner) and imports neither the CUDA
binding nor the CPU oracle, so that both sides can be fed from it.

The five workloads stand in for the paper's agentic rollout traces (Section 2.2:
a small share of very long, tool-bloated trajectories dominates rollout time;
Section 7 "Setup": lengths up to 40,960 tokens).  None of the paper's datasets is
used; only the shape of the length distribution is.

Recipes
-------
* all random numbers come from ``numpy.random.Generator(PCG64(seed))``;
* order of draws: sequence lengths, then ``permutation(pool)`` for the block
  tables, then (host generation only) q, K, V values;
* lognormal lengths: ``clip(floor(median * exp(sigma * Z) + 0.5), 1, cap)``;
* uniform lengths: integers, both ends included;
* pool size where the workload does not fix it: ``need + max(1, need // 8)``
  pages, ``need`` = sum over sequences of ``ceil(L / page_size)``;
* block tables: the first ``need`` entries of ``permutation(pool)`` cut into rows
  in batch order, unused entries ``-1``;
* values: float32 draw, rounded to bf16 with round-to-nearest-even; everything
  that must not influence a result (slots past the end of a sequence, pages no
  sequence owns) is filled with a poison value.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
from numpy.random import Generator, PCG64

PAGE_SIZE = 16
POISON_F32 = np.float32(1.0e30)  # finite in bf16; any read of it wrecks a result visibly


# --------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> float32, exact."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- workload table
@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    values: str            # "normal" | "uniform"
    lengths: str           # recipe key, see draw_seq_lens
    pool_pages: int = 0    # 0 = need + max(1, need // 8)
    steps: int = 1         # successive steps with fresh lengths (seed = step index)
    page_size: int = PAGE_SIZE
    params: dict = field(default_factory=dict)


WORKLOADS = {
    # the five workloads, in the order the benchmark lists them: 0
    "tiny": Workload("tiny", 4, 4, 1, 64, "uniform", "fixed", pool_pages=64,
                     params={"lens": [1, 7, 64, 300]}),
    # 1
    "lognormal_b64": Workload("lognormal_b64", 64, 32, 8, 128, "normal", "lognormal",
                              params={"median": [1024], "sigma": 0.8, "cap": 8192}),
    # 2
    "longtail_mix_b256": Workload("longtail_mix_b256", 256, 32, 8, 128, "normal", "mix",
                                  params={"short": (512, 4096), "long": (16384, 32768), "long_frac": 0.1}),
    # 3
    "straggler_b8": Workload("straggler_b8", 8, 64, 8, 128, "normal", "fixed",
                             params={"lens": [32768] * 8}),
    # 4
    "shift_b128": Workload("shift_b128", 128, 40, 8, 128, "normal", "lognormal", pool_pages=262144, steps=3,
                           params={"median": [1024, 2048, 4096], "sigma": 1.0, "cap": 32768}),
}
WORKLOAD_ORDER = ["tiny", "lognormal_b64", "longtail_mix_b256", "straggler_b8", "shift_b128"]


def draw_seq_lens(w: Workload, rng: Generator, step: int = 0) -> np.ndarray:
    """Sequence lengths (int32[batch]) for one step, drawn from ``rng``."""
    p = w.params
    if w.lengths == "fixed":
        lens = np.asarray(p["lens"], dtype=np.int64)
    elif w.lengths == "lognormal":
        z = rng.standard_normal(w.batch)
        med = p["median"][step]
        lens = np.clip(np.floor(med * np.exp(p["sigma"] * z) + 0.5), 1, p["cap"]).astype(np.int64)
    elif w.lengths == "mix":
        n_long = int(round(p["long_frac"] * w.batch))
        a = rng.integers(p["short"][0], p["short"][1] + 1, w.batch - n_long)
        b = rng.integers(p["long"][0], p["long"][1] + 1, n_long)
        lens = np.concatenate([a, b])[rng.permutation(w.batch)]
    else:
        raise ValueError(w.lengths)
    assert lens.shape == (w.batch,)
    return lens.astype(np.int32)


def pages_needed(seq_lens: np.ndarray, page_size: int = PAGE_SIZE) -> np.ndarray:
    return (seq_lens.astype(np.int64) + page_size - 1) // page_size


def draw_block_table(seq_lens: np.ndarray, pool_pages: int, rng: Generator,
                     page_size: int = PAGE_SIZE, ld: int | None = None) -> tuple[np.ndarray, int]:
    """Scatter the sequences' pages over the pool.  Returns (int32[B, ld], pool_pages)."""
    npg = pages_needed(seq_lens, page_size)
    need = int(npg.sum())
    if pool_pages <= 0:
        pool_pages = need + max(1, need // 8)
    assert need <= pool_pages
    perm = rng.permutation(pool_pages)[:need]
    if ld is None:
        ld = max(1, int(npg.max()) if len(npg) else 1)
    bt = np.full((len(seq_lens), ld), -1, dtype=np.int32)
    pos = 0
    for b, n in enumerate(npg):
        bt[b, :n] = perm[pos:pos + n]
        pos += n
    return bt, pool_pages


@dataclass
class Layout:
    """Metadata of one step: who owns which page.  No values."""
    workload: Workload
    step: int
    seed: int
    seq_lens: np.ndarray      # int32[B]
    block_table: np.ndarray   # int32[B, ld]
    pool_pages: int

    @property
    def total_tokens(self) -> int:
        return int(self.seq_lens.astype(np.int64).sum())

    @property
    def kv_bytes(self) -> int:
        """Algorithmic bytes of one step: K and V of every cached token, bf16, exact token count."""
        w = self.workload
        return self.total_tokens * w.num_kv_heads * w.head_dim * 2 * 2


def make_layout(name: str, step: int = 0, seed: int | None = None) -> tuple[Layout, Generator]:
    """Lengths and block table of ``name`` at ``step``; also returns the generator,
    positioned after those draws, for host-side value generation."""
    w = WORKLOADS[name]
    if seed is None:
        seed = step if w.steps > 1 else 0
    rng = Generator(PCG64(seed))
    lens = draw_seq_lens(w, rng, step)
    bt, pool = draw_block_table(lens, w.pool_pages, rng, w.page_size)
    return Layout(w, step, seed, lens, bt, pool), rng


# --------------------------------------------------------------------------- host values
def _draw_bf16(rng: Generator, shape, kind: str) -> np.ndarray:
    if kind == "normal":
        x = rng.standard_normal(shape, dtype=np.float32)
    elif kind == "uniform":
        x = rng.uniform(-1.0, 1.0, shape).astype(np.float32)
    else:
        raise ValueError(kind)
    return f32_to_bf16_bits(x)


def poison_unused(k_pages: np.ndarray, v_pages: np.ndarray, seq_lens: np.ndarray,
                  block_table: np.ndarray, page_size: int = PAGE_SIZE) -> None:
    """Overwrite, in place, every slot no sequence owns (HND pools: [page, head, slot, d])."""
    pool = k_pages.shape[0]
    keep = np.zeros((pool, page_size), dtype=bool)
    for b, L in enumerate(seq_lens):
        L = int(L)
        for i in range((L + page_size - 1) // page_size):
            n = min(page_size, L - i * page_size)
            keep[block_table[b, i], :n] = True
    pk = f32_to_bf16_bits(np.array([POISON_F32]))[0]
    nk = f32_to_bf16_bits(np.array([-POISON_F32]))[0]
    mask = ~keep  # [pool, slot]
    for arr, val in ((k_pages, pk), (v_pages, nk)):
        view = arr.transpose(0, 2, 1, 3)  # [page, slot, head, d]
        view[mask] = val


def make_host_inputs(name: str, step: int = 0, seed: int | None = None, poison: bool = True):
    """Whole workload on the host as bf16 bit patterns (uint16).  Meant for the small
    workloads; the large ones fill their pools on the device (see ``fill_device_pools``).

    Returns (layout, q[B,Hq,d], k_pages[P,Hkv,page,d], v_pages[P,Hkv,page,d]).
    """
    lay, rng = make_layout(name, step, seed)
    w = lay.workload
    q = _draw_bf16(rng, (w.batch, w.num_q_heads, w.head_dim), w.values)
    shape = (lay.pool_pages, w.num_kv_heads, w.page_size, w.head_dim)
    k = _draw_bf16(rng, shape, w.values)
    v = _draw_bf16(rng, shape, w.values)
    if poison:
        poison_unused(k, v, lay.seq_lens, lay.block_table, w.page_size)
    return lay, q, k, v


def random_case(seed: int, batch: int, num_q_heads: int, num_kv_heads: int, head_dim: int,
                seq_lens, values: str = "normal", spare_pages: int = 3, poison: bool = True,
                page_size: int = PAGE_SIZE):
    """Ad-hoc case with given lengths (used by edge-case tests)."""
    rng = Generator(PCG64(seed))
    lens = np.asarray(seq_lens, dtype=np.int32)
    assert lens.shape == (batch,)
    need = int(pages_needed(lens, page_size).sum())
    bt, pool = draw_block_table(lens, need + spare_pages, rng, page_size)
    q = _draw_bf16(rng, (batch, num_q_heads, head_dim), values)
    shape = (pool, num_kv_heads, page_size, head_dim)
    k = _draw_bf16(rng, shape, values)
    v = _draw_bf16(rng, shape, values)
    if poison:
        poison_unused(k, v, lens, bt, page_size)
    return lens, bt, q, k, v


# --------------------------------------------------------------------------- device values
def fill_device_pools(layout: Layout, device, seed: int | None = None, chunk_pages: int = 8192,
                      poison: bool = True):
    """Fill q and the K/V pools on the device with a seeded torch generator (the large
    workloads hold up to 2 x 8.6 GB of pool, too slow to draw on the host).

    Every page is filled with N(0,1) (or U[-1,1]) bf16 values; with ``poison`` the slots past
    the end of a sequence in its last page are then overwritten with the poison value (see
    ``poison_tails``).  Returns torch bf16 tensors (q[B,Hq,d], k_pages[P,Hkv,page,d],
    v_pages[P,Hkv,page,d]).
    """
    import torch

    w = layout.workload
    gen = torch.Generator(device=device)
    gen.manual_seed(1_000_003 * (layout.seed if seed is None else seed) + 17)

    def draw(shape):
        if w.values == "normal":
            return torch.randn(shape, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
        return (torch.rand(shape, generator=gen, device=device, dtype=torch.float32) * 2 - 1).to(torch.bfloat16)

    q = draw((w.batch, w.num_q_heads, w.head_dim))
    shape = (layout.pool_pages, w.num_kv_heads, w.page_size, w.head_dim)
    k = torch.empty(shape, device=device, dtype=torch.bfloat16)
    v = torch.empty(shape, device=device, dtype=torch.bfloat16)
    for t in (k, v):
        for p0 in range(0, layout.pool_pages, chunk_pages):
            p1 = min(layout.pool_pages, p0 + chunk_pages)
            t[p0:p1] = draw((p1 - p0,) + shape[1:])
    if poison:
        poison_tails(layout, k, v)
    return q, k, v


E4M3_NAN = 0x7F  # the poison of an 8-bit cache: slots past the end of a sequence hold NaN codes


def random_case_e4m3(seed: int, batch: int, num_q_heads: int, num_kv_heads: int, head_dim: int, seq_lens,
                     spare_pages: int = 3, poison: bool = True, page_size: int = PAGE_SIZE, max_exp_field: int = 8):
    """Ad-hoc case with an 8-bit KV cache: q as bf16 bits, K and V as E4M3 codes drawn as bit fields (sign,
    exponent field 0..max_exp_field, mantissa: magnitudes below 2^(max_exp_field - 6), no NaN codes), so that
    no float arithmetic is involved in making them.  Returns (lens, block_table, q, k_codes, v_codes)."""
    rng = Generator(PCG64(seed))
    lens = np.asarray(seq_lens, dtype=np.int32)
    assert lens.shape == (batch,)
    need = int(pages_needed(lens, page_size).sum())
    bt, pool = draw_block_table(lens, need + spare_pages, rng, page_size)
    q = _draw_bf16(rng, (batch, num_q_heads, head_dim), "normal")
    shape = (pool, num_kv_heads, page_size, head_dim)

    def codes():
        sign = rng.integers(0, 2, size=shape, dtype=np.uint8)
        expo = rng.integers(0, max_exp_field + 1, size=shape, dtype=np.uint8)
        mant = rng.integers(0, 8, size=shape, dtype=np.uint8)
        return (sign << 7) | (expo << 3) | mant

    k, v = codes(), codes()
    if poison:
        keep = np.zeros((pool, page_size), dtype=bool)
        for b in range(batch):
            L = int(lens[b])
            for t0 in range(0, L, page_size):
                keep[bt[b, t0 // page_size], : min(page_size, L - t0)] = True
        dead = ~keep
        k[dead[:, None, :, None] & np.ones(shape, dtype=bool)] = E4M3_NAN
        v[dead[:, None, :, None] & np.ones(shape, dtype=bool)] = E4M3_NAN | 0x80
    return lens, bt, q, k, v


def poison_tails(layout: Layout, k, v):
    """Overwrite the slots past the end of every sequence's last page (device HND pools) with the
    poison value.  Returns what was there, for ``restore_tails``: a multi-step workload reuses the
    pool with a new page placement, where those slots may hold live tokens."""
    w = layout.workload
    lens = layout.seq_lens.astype(np.int64)
    rem = lens % w.page_size
    saved = []
    for b in np.nonzero((rem != 0) & (lens > 0))[0]:
        pg = int(layout.block_table[b, (int(lens[b]) - 1) // w.page_size])
        r = int(rem[b])
        saved.append((pg, r, k[pg, :, r:, :].clone(), v[pg, :, r:, :].clone()))
        k[pg, :, r:, :] = float(POISON_F32)
        v[pg, :, r:, :] = -float(POISON_F32)
    return saved


def restore_tails(saved, k, v) -> None:
    for pg, r, ks, vs in saved:
        k[pg, :, r:, :] = ks
        v[pg, :, r:, :] = vs
