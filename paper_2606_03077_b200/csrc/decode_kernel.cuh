// Split-KV decode kernel (step D) for sm_100a.
//
// A work unit is one work item of the plan (a chunk [kv_begin, kv_end) of one sequence) for one KV
// head and all G query heads that share it.  The kernel works in tiles of 16 tokens: a page of 16, 32
// or 64 tokens is 1, 2 or 4 tiles ("page" below means such a tile).  Inside a thread block every warp
// owns a private ring of shared-memory stages and takes the unit's tiles warp, warp+NW, warp+2NW, ...:
//
//   lane 0 : page id -> two tiled TMA loads per tensor (K and V page, 128-byte swizzle) that
//            complete on the stage's mbarrier; up to STAGES pages per warp are in flight
//   warp   : S^T[16 tokens x 8 heads]  = K_page . Q^T       mma.sync m16n8k16 bf16 -> fp32
//            online softmax in fp32 (running max m and sum l per head, base-2 exponent)
//            O^T[d x 8 heads]         += V_page^T . P^T     P as two bf16 terms (head + rounding residue)
//
// Tokens are the M side of the tiles, the (padded) head group the N side, so a group of up to
// 8 heads costs one 8-wide tile and nothing is wasted on padding rows; with 9 to 16 rows of q per KV
// head (a wider group, or several query tokens) the rows of q take the M side instead (process_page_rows).
// The kernel is bound by the HBM read of K and V: 2 * head_dim * 2 bytes per token per KV head,
// 4 * G * head_dim flop.
//
// The warps never synchronise with each other while they stream pages; they merge their (m, l, O)
// in shared memory once per unit, in warp order, so results are bit-reproducible.
//
// Step C can run inside decode_kernel: every block of a split sequence bumps a per-(sequence, KV
// head) counter after publishing its partial result, and the block that arrives last merges all
// partials in chunk order (the same arithmetic, in the same order, as the stand-alone combine kernel).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "combine_kernel.cuh"
#include "plan_layout.hpp"

namespace libra {

struct DecodeParams {
  const __nv_bfloat16* q;
  const int32_t* block_table;
  const int32_t* seq_lens;
  __nv_bfloat16* out;
  float* lse_out;        // [B][rows] natural-log sum of exponentials of every row of q, or null
  const int4* entries;   // work items then empty-sequence entries in device memory, or null: in `pp`
  const int32_t* dev_counts;  // device-side plan: the counts below are read from here (null = host plan)
  float* partial_o;      // [slot][Hq][D]
  float* partial_lse;    // [slot][Hq]
  uint32_t* error_word;
  int32_t* counters;      // [batch][Hkv] arrival counters of split sequences (zero between launches)
  int64_t num_pages;
  int32_t num_q_heads;    // rows of q / out per sequence: query tokens x query heads
  int32_t num_kv_heads;
  int32_t group;          // G
  int32_t q_len;          // Tq: query tokens per sequence (the last Tq tokens of the cache are theirs); usually 1
  int32_t hq;             // query heads of the model (num_q_heads = q_len * hq)
  int32_t cols;           // q_len * G: rows of q that share one KV head = columns of a unit's score tile
  int32_t block_table_ld;
  float scale_log2;       // sm_scale * log2(e) (times the key scale of an 8-bit cache)
  float v_scale;          // value scale of an 8-bit cache; 1 for a bf16 cache
  int32_t pos_head;       // coordinate slot (1..3) of the head / page / token dimension in the tensor maps
  int32_t pos_page;
  int32_t pos_token;
  int32_t tile_shift;     // log2(page_size / 16): a page holds 1, 2 or 4 tiles of 16 tokens
  int32_t num_items;
  int32_t num_units;      // work items x KV heads
  int32_t num_empty;      // empty sequences whose output row this launch zeroes
  int32_t fused_combine;  // 1: the last block of a split sequence merges its partials (step C) itself
  int32_t early_prefetch; // 1: block-table walk and first copies of old tokens start before the grid dependency wait
  int32_t l2_warmup;      // 1: first-wave blocks ask for their first tiles to be brought into L2 before that wait
  // KV append fused into the step (null k_new = off): the K and V rows of the newest q_len tokens, [B, q_len, Hkv, D]
  // in the cache's element type, are written into their slots of the sequence's last page(s), in the pools and in the
  // staged tiles
  const void* k_new;
  const void* v_new;
  void* k_pool;
  void* v_pool;
  int64_t stride_page, stride_head, stride_token;  // pool strides in elements
};

namespace dev {

constexpr uint32_t kWaitLimit = 1u << 20;  // tries of a bounded wait on a copy barrier (each suspends <= ~2 us)
constexpr uint32_t kWaitHintNs = 2000;
// The running maximum of a column is raised only when a tile's maximum exceeds it by more than this many powers of
// two (and then every column of the warp is brought up to date): between raises the probabilities may reach
// 2^kMaxSlack instead of 1, which bf16 / fp16 and the fp32 sums hold with the same relative precision, and the
// accumulators are not rescaled tile after tile (a warp sees every NW-th tile of a unit, so its maximum keeps
// growing for most of a short unit).
#ifndef LIBRA_MAX_SLACK
#define LIBRA_MAX_SLACK 8.0f
#endif
constexpr float kMaxSlack = LIBRA_MAX_SLACK;
// 1: the probabilities of a bf16 cache go to the tensor core as two bf16 terms (see process_page)
#ifndef LIBRA_SPLIT_P
#define LIBRA_SPLIT_P 1
#endif
// 1: with 9 - 16 score columns per KV head (bf16 cache) the columns are the M side of the tiles (process_page_rows)
#ifndef LIBRA_ROWS_LAYOUT
#define LIBRA_ROWS_LAYOUT 1
#endif

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kWaitHintNs)
      : "memory");
  return ok != 0;
}
// Returns false if the barrier did not complete within `limit` tries.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit = kWaitLimit) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  return false;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

// L2 policy for data that is read once: pages of K and V are streamed, never reused, so they should be the first
// to leave L2 and not push out what IS reused (q, block tables, the plan, partial results).
// Measured: 57.7 -> 56.2 us per step on the headline workload, 0.5 - 1.5 % on the others.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}

// Tiled 4-D TMA load global -> shared (one destination block only) with an L2 cache policy, completing on an mbarrier of this block.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      :
      : "r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}

// Ask for one box of a tiled tensor to be brought into L2 (no destination, nothing to wait for).
__device__ __forceinline__ void tma_prefetch_l2_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3, uint64_t policy) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile.L2::cache_hint [%0, {%1, %2, %3, %4}], %5;"
               :
               : "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
               : "memory");
}

// A 32-bit load that goes to L2, not through this SM's L1 (for memory another kernel may still be writing).
__device__ __forceinline__ int32_t ld_cg_s32(const int32_t* ptr) {
  int32_t v;
  asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}

__device__ __forceinline__ uint32_t sm_count() {
  uint32_t n;
  asm volatile("mov.u32 %0, %%nsmid;" : "=r"(n));
  return n;
}

// Pull a tensor map (a kernel parameter) into the descriptor cache ahead of its first use.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr)
               : "memory");
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
// D(16x8, fp32) += A(16x16 bf16, row) * B(16x8 bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Same shape with fp16 operands (used with an 8-bit cache, whose codes convert to fp16 exactly).
__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Four E4M3 codes -> two fp16 pairs: lo = codes 0, 1; hi = codes 2, 3 (exact: E4M3 is a subset of fp16).
__device__ __forceinline__ void cvt_e4m3x4(uint32_t x, uint32_t& lo, uint32_t& hi) {
  asm("{\n\t.reg .b16 a, b;\n\t"
      "mov.b32 {a, b}, %2;\n\t"
      "cvt.rn.f16x2.e4m3x2 %0, a;\n\t"
      "cvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
      : "=r"(lo), "=r"(hi)
      : "r"(x));
}
__device__ __forceinline__ uint32_t byte_perm_3120(uint32_t x) {
  uint32_t d;
  asm("prmt.b32 %0, %1, 0, 0x3120;" : "=r"(d) : "r"(x));
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Byte offset of 16-byte chunk c16 of row r inside a [D/64][16][128 B] tile with 128-byte swizzle.
__device__ __forceinline__ uint32_t tile_off(int r, int c16) {
  return uint32_t(((c16 >> 3) << 11) + (r << 7) + ((((c16 & 7) ^ (r & 7))) << 4));
}

// One decoded work unit as a warp sees it.
struct Unit {
  int b, kvh, kv_begin, kv_end, slot, chunk_j, n_chunks;
  int n_it;       // pages of the unit this warp takes
  int first_page; // index of the unit's first page in the sequence's block-table row
};

template <int NW>
__device__ __forceinline__ Unit decode_unit(const int4 item, int kvh, int warp) {
  Unit u;
  u.b = item.x & (plan_layout::kMaxBatch - 1);
  u.chunk_j = (item.x >> plan_layout::kChunkShift) & 63;
  u.n_chunks = item.x >> plan_layout::kCountShift;
  u.kv_begin = item.y;
  u.kv_end = item.z;
  u.slot = item.w;  // < 0: the sequence is not split, write bf16 `out` directly
  u.kvh = kvh;
  const int n_pages = (u.kv_end - u.kv_begin + 15) >> 4;
  u.first_page = u.kv_begin >> 4;
  u.n_it = (n_pages > warp) ? (n_pages - warp + NW - 1) / NW : 0;
  return u;
}

// Column c of a unit (KV head kvh) is query token c / G, head kvh * G + c % G of that token; q and out are
// [B, q_len, hq, d], so the row within a sequence is:
__device__ __forceinline__ int col_row(const DecodeParams& p, int kvh, int c) {
  if (p.q_len == 1) return kvh * p.group + c;   // the usual case, without the division
  const int i = c / p.group;
  return i * p.hq + kvh * p.group + (c - i * p.group);
}

// Q^T fragments (B operand: k = dims, n = columns); columns >= cols are zero.
template <int D, int NT>
__device__ __forceinline__ void load_q_frags(uint32_t (&qf)[NT][D / 16][2], const DecodeParams& p, int b, int kvh,
                                             int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const int head = nt * 8 + g;
    const bool live = head < p.cols;
    const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
        p.q + (int64_t(b) * p.num_q_heads + col_row(p, kvh, live ? head : 0)) * D);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      qf[nt][kk][0] = live ? __ldg(qrow + 8 * kk + t) : 0u;
      qf[nt][kk][1] = live ? __ldg(qrow + 8 * kk + t + 4) : 0u;
    }
  }
}

// The running maximum starts at a huge negative finite value, not -inf: a column all of whose tokens so far were
// masked (score -inf) then keeps m finite, so m_old - m_new = 0 and score - m = -inf give the factors 1 and 0
// that leave its zeros alone, with no special case.  Real scores are nowhere near it.
constexpr float kNegBig = -1.0e30f;

// Running softmax state of one warp: columns 2t, 2t+1 of every 8-wide tile.
template <int D, int NT>
struct WarpAcc {
  float m[NT][2], l[NT][2];
  float acc[NT][D / 16][4];
  __device__ __forceinline__ void reset() {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      m[nt][0] = m[nt][1] = kNegBig;
      l[nt][0] = l[nt][1] = 0.f;
#pragma unroll
      for (int mt = 0; mt < D / 16; ++mt) acc[nt][mt][0] = acc[nt][mt][1] = acc[nt][mt][2] = acc[nt][mt][3] = 0.f;
    }
  }
};

// One page (16 tokens) of one KV head: scores, online softmax update, PV accumulation.
// kt / vt: shared-memory addresses of the K and V tiles; v_gen: generic pointer to the V tile.
// n_valid: tokens of the tile inside the unit's chunk.  n_common: tokens of the tile that EVERY column sees
// (< n_valid only where several query tokens end at different positions); when it is < 16 the columns are
// masked one by one: column (nt, e) of this thread sees the first len_rel - cut[nt][e] tokens of the tile.
template <int D, int NT>
__device__ __forceinline__ void process_page(WarpAcc<D, NT>& st, const uint32_t (&qf)[NT][D / 16][2], uint32_t kt,
                                             uint32_t vt, uint8_t* v_gen, int n_valid, float scale_log2, int lane,
                                             int n_common, int len_rel, const int (&cut)[NT][2]) {
  constexpr int KS = D / 16;
  const int g = lane >> 2;
  const int k_row = lane & 15, k_sel = lane >> 4;
  const int v_row = (lane & 7) + ((lane >> 4) << 3), v_sel = (lane >> 3) & 1;

  if (n_valid < 16) {
    // rows past the end may hold anything, NaN included: clear them in V so that 0 * garbage cannot leak
    for (int i = lane; i < (16 - n_valid) * (D / 8); i += 32) {
      const int r = n_valid + i / (D / 8);
      const int c16 = i % (D / 8);
      *reinterpret_cast<uint4*>(v_gen + ((c16 >> 3) << 11) + (r << 7) + ((c16 & 7) << 4)) = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async();  // these generic writes come before the next TMA write into this stage
    __syncwarp();
  }

  // ---- S^T = K . Q^T  (two accumulator sets to halve the dependent chain)
  float sc[NT][4], sc2[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
    sc2[nt][0] = sc2[nt][1] = sc2[nt][2] = sc2[nt][3] = 0.f;
  }
#pragma unroll
  for (int kk = 0; kk < KS; ++kk) {
    uint32_t a[4];
    ldsm_x4(a, kt + tile_off(k_row, 2 * kk + k_sel));
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      if (kk & 1) mma_bf16(sc2[nt], a, qf[nt][kk][0], qf[nt][kk][1]);
      else mma_bf16(sc[nt], a, qf[nt][kk][0], qf[nt][kk][1]);
    }
  }

  // ---- online softmax; this thread holds tokens g, g+8 for heads 2t, 2t+1
  uint32_t pb[NT][2];
  bool grew = false;
  float m_new[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) sc[nt][e] = (sc[nt][e] + sc2[nt][e]) * scale_log2;
    if (n_common < 16) {
      const int nv0 = min(n_valid, len_rel - cut[nt][0]), nv1 = min(n_valid, len_rel - cut[nt][1]);
      if (g >= nv0) sc[nt][0] = -INFINITY;
      if (g >= nv1) sc[nt][1] = -INFINITY;
      if (g + 8 >= nv0) sc[nt][2] = -INFINITY;
      if (g + 8 >= nv1) sc[nt][3] = -INFINITY;
    }
    float mx0 = fmaxf(sc[nt][0], sc[nt][2]);
    float mx1 = fmaxf(sc[nt][1], sc[nt][3]);
#pragma unroll
    for (int off = 4; off <= 16; off <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
    }
    m_new[nt][0] = fmaxf(st.m[nt][0], mx0);
    m_new[nt][1] = fmaxf(st.m[nt][1], mx1);
    grew = grew || (mx0 > st.m[nt][0] + kMaxSlack) || (mx1 > st.m[nt][1] + kMaxSlack);
  }
  if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float f0 = ex2(st.m[nt][0] - m_new[nt][0]);  // first page: 2^(-huge) = 0 on zeros
      const float f1 = ex2(st.m[nt][1] - m_new[nt][1]);
      st.l[nt][0] *= f0;
      st.l[nt][1] *= f1;
#pragma unroll
      for (int mt = 0; mt < KS; ++mt) {
        st.acc[nt][mt][0] *= f0;
        st.acc[nt][mt][1] *= f1;
        st.acc[nt][mt][2] *= f0;
        st.acc[nt][mt][3] *= f1;
      }
      st.m[nt][0] = m_new[nt][0];
      st.m[nt][1] = m_new[nt][1];
    }
  }
#if LIBRA_SPLIT_P
  uint32_t pr[NT][2];   // what rounding P to bf16 lost, as a second bf16 operand
#endif
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const float p0 = ex2(sc[nt][0] - st.m[nt][0]);
    const float p1 = ex2(sc[nt][1] - st.m[nt][1]);
    const float p2 = ex2(sc[nt][2] - st.m[nt][0]);
    const float p3 = ex2(sc[nt][3] - st.m[nt][1]);
    const __nv_bfloat162 lo = __floats2bfloat162_rn(p0, p1);  // token g   : heads 2t, 2t+1
    const __nv_bfloat162 hi = __floats2bfloat162_rn(p2, p3);  // token g+8
    const uint32_t ulo = *reinterpret_cast<const uint32_t*>(&lo);
    const uint32_t uhi = *reinterpret_cast<const uint32_t*>(&hi);
    const float r0 = __uint_as_float(ulo << 16), r1 = __uint_as_float(ulo & 0xffff0000u);
    const float r2 = __uint_as_float(uhi << 16), r3 = __uint_as_float(uhi & 0xffff0000u);
#if LIBRA_SPLIT_P
    // P = head + tail, both bf16: the tail carries the 8 bits that the head's rounding dropped, so the weights the
    // tensor core applies are P to 2^-17 instead of 2^-9 (the tensor pipe is all but idle in this kernel; without the
    // tail the rounding of P is the largest error of the whole step, ~0.2 % of a row's rms)
    const __nv_bfloat162 lo2 = __floats2bfloat162_rn(p0 - r0, p1 - r1);
    const __nv_bfloat162 hi2 = __floats2bfloat162_rn(p2 - r2, p3 - r3);
    pr[nt][0] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&lo2));
    pr[nt][1] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&hi2));
    st.l[nt][0] += p0 + p2;
    st.l[nt][1] += p1 + p3;
#else
    // the denominator sums exactly the probabilities the tensor core will see
    st.l[nt][0] += r0 + r2;
    st.l[nt][1] += r1 + r3;
#endif
    pb[nt][0] = movmatrix_trans(ulo);  // head g : tokens 2t, 2t+1
    pb[nt][1] = movmatrix_trans(uhi);  // head g : tokens 2t+8, 2t+9
  }

  // ---- O^T += V^T . P^T
#pragma unroll
  for (int mt = 0; mt < KS; ++mt) {
    uint32_t a[4];
    ldsm_x4_trans(a, vt + tile_off(v_row, 2 * mt + v_sel));
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      mma_bf16(st.acc[nt][mt], a, pb[nt][0], pb[nt][1]);
#if LIBRA_SPLIT_P
      mma_bf16(st.acc[nt][mt], a, pr[nt][0], pr[nt][1]);
#endif
    }
  }
}

// ---- 9 to 16 score columns per KV head: the columns on the M side --------------------------------------
// With more than 8 rows of q per KV head (a wide head group, or several query tokens) the tile shapes turn round: the
// 16 rows of q are the M side of every mma, so
//   S[16 cols x 16 tokens]  = Q . K_page^T      A = Q fragments (registers), B = K rows as ldmatrix delivers them
//   O[16 cols x d]         += P . V_page        A = P, which is S's accumulator layout as it stands (no register
//                                               transposes), B = V by ldmatrix.trans
// A thread holds rows g and g + 8 of S: one running maximum and sum per row (two per thread instead of four), and a
// row's maximum is two shuffles away (over the four lanes of a quad) instead of three.  The state lives in the same
// WarpAcc<D, 2>: m[0][0] / m[0][1] (and l) are rows g / g + 8, acc[n / (D/16)][n % (D/16)] is the 8-dim slice n of O with
// c0, c1 = row g, dims 8n + 2t, + 1 and c2, c3 = row g + 8.

// Q fragments as the A operand, kept in qf[NT = 2][D / 16][2]: {qf[0][kk][0], qf[0][kk][1], qf[1][kk][0], qf[1][kk][1]}
// = {row g dims 16kk + 2t.., row g + 8 same dims, row g dims 16kk + 8 + 2t.., row g + 8}; rows >= cols are zero.
template <int D>
__device__ __forceinline__ void load_q_frags_rows(uint32_t (&qf)[2][D / 16][2], const DecodeParams& p, int b, int kvh,
                                                  int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int hi = 0; hi < 2; ++hi) {
    const int row = g + 8 * hi;
    const bool live = row < p.cols;
    const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
        p.q + (int64_t(b) * p.num_q_heads + col_row(p, kvh, live ? row : 0)) * D);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      qf[0][kk][hi] = live ? __ldg(qrow + 8 * kk + t) : 0u;
      qf[1][kk][hi] = live ? __ldg(qrow + 8 * kk + t + 4) : 0u;
    }
  }
}

// One page (16 tokens) of one KV head in that layout; same contract as process_page, `cut` per row: cut[0][0] for row
// g, cut[0][1] for row g + 8.
template <int D>
__device__ __forceinline__ void process_page_rows(WarpAcc<D, 2>& st, const uint32_t (&qf)[2][D / 16][2], uint32_t kt,
                                                  uint32_t vt, uint8_t* v_gen, int n_valid, float scale_log2, int lane,
                                                  int n_common, int len_rel, const int (&cut)[2][2]) {
  constexpr int KS = D / 16;
  const int t = lane & 3;
  const int k_row = lane & 15, k_sel = lane >> 4;
  const int v_row = (lane & 7) + ((lane >> 4) << 3), v_sel = (lane >> 3) & 1;

  if (n_valid < 16) {
    // rows past the end may hold anything, NaN included: clear them in V so that 0 * garbage cannot leak
    for (int i = lane; i < (16 - n_valid) * (D / 8); i += 32) {
      const int r = n_valid + i / (D / 8);
      const int c16 = i % (D / 8);
      *reinterpret_cast<uint4*>(v_gen + ((c16 >> 3) << 11) + (r << 7) + ((c16 & 7) << 4)) = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async();  // these generic writes come before the next TMA write into this stage
    __syncwarp();
  }

  // ---- S = Q . K^T: n-tile 0 = tokens 0 - 7, n-tile 1 = tokens 8 - 15; even and odd k-steps in separate accumulators
  float sc[2][4], sc2[2][4];
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
    sc2[nt][0] = sc2[nt][1] = sc2[nt][2] = sc2[nt][3] = 0.f;
  }
#pragma unroll
  for (int kk = 0; kk < KS; ++kk) {
    uint32_t r[4];   // {tokens 0-7 dims lo, tokens 8-15 dims lo, tokens 0-7 dims hi, tokens 8-15 dims hi} of k-step kk
    ldsm_x4(r, kt + tile_off(k_row, 2 * kk + k_sel));
    const uint32_t a[4] = {qf[0][kk][0], qf[0][kk][1], qf[1][kk][0], qf[1][kk][1]};
    if (kk & 1) {
      mma_bf16(sc2[0], a, r[0], r[2]);
      mma_bf16(sc2[1], a, r[1], r[3]);
    } else {
      mma_bf16(sc[0], a, r[0], r[2]);
      mma_bf16(sc[1], a, r[1], r[3]);
    }
  }

  // ---- online softmax; this thread holds rows g (e = 0, 1) and g + 8 (e = 2, 3) at tokens 8 nt + 2t, + 1
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) sc[nt][e] = (sc[nt][e] + sc2[nt][e]) * scale_log2;
  }
  if (n_common < 16) {
    const int nv0 = min(n_valid, len_rel - cut[0][0]), nv1 = min(n_valid, len_rel - cut[0][1]);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int tok = 8 * nt + 2 * t;
      if (tok >= nv0) sc[nt][0] = -INFINITY;
      if (tok + 1 >= nv0) sc[nt][1] = -INFINITY;
      if (tok >= nv1) sc[nt][2] = -INFINITY;
      if (tok + 1 >= nv1) sc[nt][3] = -INFINITY;
    }
  }
  float mx0 = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1]));
  float mx1 = fmaxf(fmaxf(sc[0][2], sc[0][3]), fmaxf(sc[1][2], sc[1][3]));
#pragma unroll
  for (int off = 1; off <= 2; off <<= 1) {
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
  }
  const bool grew = (mx0 > st.m[0][0] + kMaxSlack) || (mx1 > st.m[0][1] + kMaxSlack);
  if (__any_sync(0xffffffffu, grew)) {
    const float m0 = fmaxf(st.m[0][0], mx0), m1 = fmaxf(st.m[0][1], mx1);
    const float f0 = ex2(st.m[0][0] - m0), f1 = ex2(st.m[0][1] - m1);
    st.l[0][0] *= f0;
    st.l[0][1] *= f1;
#pragma unroll
    for (int n = 0; n < D / 8; ++n) {
      st.acc[n / KS][n % KS][0] *= f0;
      st.acc[n / KS][n % KS][1] *= f0;
      st.acc[n / KS][n % KS][2] *= f1;
      st.acc[n / KS][n % KS][3] *= f1;
    }
    st.m[0][0] = m0;
    st.m[0][1] = m1;
  }
  // P as the A operand of the second product: {row g tokens 2t.., row g + 8 tokens 2t.., row g tokens 8 + 2t.., row g + 8}
  uint32_t pa[4], pr[4];
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    const float p0 = ex2(sc[nt][0] - st.m[0][0]), p1 = ex2(sc[nt][1] - st.m[0][0]);
    const float p2 = ex2(sc[nt][2] - st.m[0][1]), p3 = ex2(sc[nt][3] - st.m[0][1]);
    const __nv_bfloat162 lo = __floats2bfloat162_rn(p0, p1), hi = __floats2bfloat162_rn(p2, p3);
    const uint32_t ulo = *reinterpret_cast<const uint32_t*>(&lo), uhi = *reinterpret_cast<const uint32_t*>(&hi);
    pa[2 * nt] = ulo;
    pa[2 * nt + 1] = uhi;
    // the residue of the rounding as a second bf16 term (see process_page)
    const __nv_bfloat162 lo2 = __floats2bfloat162_rn(p0 - __uint_as_float(ulo << 16), p1 - __uint_as_float(ulo & 0xffff0000u));
    const __nv_bfloat162 hi2 = __floats2bfloat162_rn(p2 - __uint_as_float(uhi << 16), p3 - __uint_as_float(uhi & 0xffff0000u));
    pr[2 * nt] = *reinterpret_cast<const uint32_t*>(&lo2);
    pr[2 * nt + 1] = *reinterpret_cast<const uint32_t*>(&hi2);
    st.l[0][0] += p0 + p1;
    st.l[0][1] += p2 + p3;
  }

  // ---- O += P . V: one ldmatrix.trans feeds two 8-dim slices
#pragma unroll
  for (int mt = 0; mt < KS; ++mt) {
    uint32_t r[4];   // {tokens 0-7 dims 16mt.., tokens 0-7 dims 16mt + 8.., tokens 8-15 dims 16mt.., tokens 8-15 dims 16mt + 8..}
    ldsm_x4_trans(r, vt + tile_off(v_row, 2 * mt + v_sel));
    float (&o0)[4] = st.acc[(2 * mt) / KS][(2 * mt) % KS];
    float (&o1)[4] = st.acc[(2 * mt + 1) / KS][(2 * mt + 1) % KS];
    mma_bf16(o0, pa, r[0], r[2]);
    mma_bf16(o1, pa, r[1], r[3]);
    mma_bf16(o0, pr, r[0], r[2]);
    mma_bf16(o1, pr, r[1], r[3]);
  }
}

// That layout's result -> shared memory, in the form merge_and_write reads: stats per row, O as [row][dim] fp32 with
// the dim index XORed with stage_swizzle(row).
template <int D>
__device__ __forceinline__ void stage_warp_result_rows(WarpAcc<D, 2>& st, float* o_sm, float* m_sm, float* l_sm, int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int off = 1; off <= 2; off <<= 1) {   // l is spread over the four lanes of a quad
    st.l[0][0] += __shfl_xor_sync(0xffffffffu, st.l[0][0], off);
    st.l[0][1] += __shfl_xor_sync(0xffffffffu, st.l[0][1], off);
  }
  if (t == 0) {
    m_sm[g] = st.m[0][0];
    m_sm[g + 8] = st.m[0][1];
    l_sm[g] = st.l[0][0];
    l_sm[g + 8] = st.l[0][1];
  }
  const int sw0 = ((g >> 1) & 3) << 3;   // = stage_swizzle(g) = stage_swizzle(g + 8)
#pragma unroll
  for (int n = 0; n < D / 8; ++n) {
    const float (&o)[4] = st.acc[n / (D / 16)][n % (D / 16)];
    const int d0 = (8 * n + 2 * t) ^ sw0;   // the XOR moves whole groups of 8 dims: the pair stays together
    *reinterpret_cast<float2*>(o_sm + g * D + d0) = make_float2(o[0], o[1]);
    *reinterpret_cast<float2*>(o_sm + (g + 8) * D + d0) = make_float2(o[2], o[3]);
  }
}

// ---- 8-bit (E4M3) cache ---------------------------------------------------------------------------
// A tile is 16 tokens x D bytes: rows of 128 bytes with the 128-byte swizzle (head_dim 128) or rows of 64 bytes
// with the 64-byte swizzle (head_dim 64).  ldmatrix moves it as 16-bit units, i.e.
// PAIRS of codes, so the fragments come out in an order of their own; sums over k and the assignment of
// output rows do not care about order as long as both operands agree:
//   scores : within a 16-dim chunk, mma k-slots (2t, 2t+1, 2t+8, 2t+9) carry dims (4t, 4t+1, 4t+2, 4t+3)
//   output : within a 16-dim chunk, mma rows (g, g+8) carry dims (2g, 2g+1)
// Codes are converted to fp16 (exact); q is converted bf16 -> fp16 (exact for |q| in [2^-14, 65504]) and P is
// rounded to fp16.  (Converting the values with integer operations instead, to unload the pipe the conversion
// instruction shares with the exponentials, measured 5-10 % slower.)

// Byte offset of 16-byte chunk c of row r in such a tile (the copy engine's swizzle: the chunk index is XORed with
// address bits 7 and up - 3 of them for 128-byte rows, 2 for 64-byte rows).
template <int D>
__device__ __forceinline__ uint32_t tile_off_fp8(int r, int c) {
  if constexpr (D == 128) return uint32_t((r << 7) + ((c ^ (r & 7)) << 4));
  else return uint32_t((r << 6) + ((c ^ ((r >> 1) & 3)) << 4));
}

// Q^T fragments in that k-order, fp16; columns >= cols are zero.
template <int D, int NT>
__device__ __forceinline__ void load_q_frags_fp8(uint32_t (&qf)[NT][D / 16][2], const DecodeParams& p, int b, int kvh,
                                                 int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const int col = nt * 8 + g;
    const bool live = col < p.cols;
    const __nv_bfloat16* qrow = p.q + (int64_t(b) * p.num_q_heads + col_row(p, kvh, live ? col : 0)) * D;
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      const uint2 raw = __ldg(reinterpret_cast<const uint2*>(qrow + 16 * kk + 4 * t));   // dims 4t .. 4t+3 of chunk kk
      const __nv_bfloat162 x01 = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
      const __nv_bfloat162 x23 = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
      const __half2 h01 = __floats2half2_rn(__low2float(x01), __high2float(x01));
      const __half2 h23 = __floats2half2_rn(__low2float(x23), __high2float(x23));
      qf[nt][kk][0] = live ? *reinterpret_cast<const uint32_t*>(&h01) : 0u;
      qf[nt][kk][1] = live ? *reinterpret_cast<const uint32_t*>(&h23) : 0u;
    }
  }
}

// One page (16 tokens) of one KV head from an E4M3 cache; same contract as process_page.
template <int D, int NT>
__device__ __forceinline__ void process_page_fp8(WarpAcc<D, NT>& st, const uint32_t (&qf)[NT][D / 16][2], uint32_t kt,
                                                 uint32_t vt, uint8_t* v_gen, int n_valid, float scale_log2, int lane,
                                                 int n_common, int len_rel, const int (&cut)[NT][2]) {
  const int g = lane >> 2;
  // ldmatrix.x4: lanes 0-7 / 8-15 give the rows (tokens 0-7 / 8-15) of 16-byte chunk c, lanes 16-31 those of chunk c+1
  const int row = (lane & 7) + ((lane >> 3) & 1) * 8;
  const int csel = lane >> 4;

  if (n_valid < 16) {
    // rows past the end may hold anything, NaN codes included: clear them in V so that 0 * garbage cannot leak
    for (int i = lane; i < (16 - n_valid) * (D / 16); i += 32) {
      const int r = n_valid + i / (D / 16);
      *reinterpret_cast<uint4*>(v_gen + r * D + ((i % (D / 16)) << 4)) = make_uint4(0, 0, 0, 0);
    }
    fence_proxy_async();  // these generic writes come before the next TMA write into this stage
    __syncwarp();
  }

  // ---- S^T = K . Q^T
  float sc[NT][4], sc2[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
    sc2[nt][0] = sc2[nt][1] = sc2[nt][2] = sc2[nt][3] = 0.f;
  }
#pragma unroll
  for (int c2 = 0; c2 < D / 32; ++c2) {
    uint32_t r[4];   // (tokens 0-7, chunk 2 c2), (tokens 8-15, chunk 2 c2), (tokens 0-7, chunk 2 c2 + 1), (tokens 8-15, chunk 2 c2 + 1)
    ldsm_x4(r, kt + tile_off_fp8<D>(row, 2 * c2 + csel));
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t a[4];
      cvt_e4m3x4(r[2 * half], a[0], a[2]);        // token g   : dims 4t, 4t+1 | 4t+2, 4t+3
      cvt_e4m3x4(r[2 * half + 1], a[1], a[3]);    // token g+8
      const int kk = 2 * c2 + half;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        if (half) mma_f16(sc2[nt], a, qf[nt][kk][0], qf[nt][kk][1]);
        else mma_f16(sc[nt], a, qf[nt][kk][0], qf[nt][kk][1]);
      }
    }
  }

  // ---- online softmax; this thread holds tokens g, g+8 for columns 2t, 2t+1
  uint32_t pb[NT][2];
  bool grew = false;
  float m_new[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) sc[nt][e] = (sc[nt][e] + sc2[nt][e]) * scale_log2;
    if (n_common < 16) {
      const int nv0 = min(n_valid, len_rel - cut[nt][0]), nv1 = min(n_valid, len_rel - cut[nt][1]);
      if (g >= nv0) sc[nt][0] = -INFINITY;
      if (g >= nv1) sc[nt][1] = -INFINITY;
      if (g + 8 >= nv0) sc[nt][2] = -INFINITY;
      if (g + 8 >= nv1) sc[nt][3] = -INFINITY;
    }
    float mx0 = fmaxf(sc[nt][0], sc[nt][2]);
    float mx1 = fmaxf(sc[nt][1], sc[nt][3]);
#pragma unroll
    for (int off = 4; off <= 16; off <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
    }
    m_new[nt][0] = fmaxf(st.m[nt][0], mx0);
    m_new[nt][1] = fmaxf(st.m[nt][1], mx1);
    grew = grew || (mx0 > st.m[nt][0] + kMaxSlack) || (mx1 > st.m[nt][1] + kMaxSlack);
  }
  if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float f0 = ex2(st.m[nt][0] - m_new[nt][0]);
      const float f1 = ex2(st.m[nt][1] - m_new[nt][1]);
      st.l[nt][0] *= f0;
      st.l[nt][1] *= f1;
#pragma unroll
      for (int mt = 0; mt < D / 16; ++mt) {
        st.acc[nt][mt][0] *= f0;
        st.acc[nt][mt][1] *= f1;
        st.acc[nt][mt][2] *= f0;
        st.acc[nt][mt][3] *= f1;
      }
      st.m[nt][0] = m_new[nt][0];
      st.m[nt][1] = m_new[nt][1];
    }
  }
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const __half2 lo = __floats2half2_rn(ex2(sc[nt][0] - st.m[nt][0]), ex2(sc[nt][1] - st.m[nt][1]));  // token g
    const __half2 hi = __floats2half2_rn(ex2(sc[nt][2] - st.m[nt][0]), ex2(sc[nt][3] - st.m[nt][1]));  // token g+8
    // the denominator sums exactly the probabilities the tensor core will see
    const float2 flo = __half22float2(lo), fhi = __half22float2(hi);
    st.l[nt][0] += flo.x + fhi.x;
    st.l[nt][1] += flo.y + fhi.y;
    pb[nt][0] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&lo));  // column g : tokens 2t, 2t+1
    pb[nt][1] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&hi));  // column g : tokens 2t+8, 2t+9
  }

  // ---- O^T += V^T . P^T
#pragma unroll
  for (int c2 = 0; c2 < D / 32; ++c2) {
    uint32_t r[4];   // transposed: this thread gets, per matrix, {token 2t: dims 2g, 2g+1 | token 2t+1: dims 2g, 2g+1}
    ldsm_x4_trans(r, vt + tile_off_fp8<D>(row, 2 * c2 + csel));
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t a[4];
      cvt_e4m3x4(byte_perm_3120(r[2 * half]), a[0], a[1]);      // dim 2g | dim 2g+1 : tokens 2t, 2t+1
      cvt_e4m3x4(byte_perm_3120(r[2 * half + 1]), a[2], a[3]);  //                    tokens 2t+8, 2t+9
      const int mt = 2 * c2 + half;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) mma_f16(st.acc[nt][mt], a, pb[nt][0], pb[nt][1]);
    }
  }
}

// A warp's unit result -> shared memory: stats m, l per head and O as [head][dim] fp32.
// kPairDims: accumulator rows (g, g+8) of a 16-dim chunk hold dims (2g, 2g+1) instead of (g, g+8).
template <int D, int NT, bool kPairDims = false>
__device__ __forceinline__ void stage_warp_result(WarpAcc<D, NT>& st, float* o_sm, float* m_sm, float* l_sm, int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
    for (int off = 4; off <= 16; off <<= 1) {  // l is spread over the 8 token lanes of each head
      st.l[nt][0] += __shfl_xor_sync(0xffffffffu, st.l[nt][0], off);
      st.l[nt][1] += __shfl_xor_sync(0xffffffffu, st.l[nt][1], off);
    }
    if (g == 0) {
      m_sm[nt * 8 + 2 * t] = st.m[nt][0];
      m_sm[nt * 8 + 2 * t + 1] = st.m[nt][1];
      l_sm[nt * 8 + 2 * t] = st.l[nt][0];
      l_sm[nt * 8 + 2 * t + 1] = st.l[nt][1];
    }
#pragma unroll
    for (int mt = 0; mt < D / 16; ++mt) {
      const int h0 = nt * 8 + 2 * t;
      const int d0 = mt * 16 + (kPairDims ? 2 * g : g);
      constexpr int kStep = kPairDims ? 1 : 8;
      // rows are D floats apart, a multiple of the 32 banks, so the four lanes that share g would hit one bank:
      // the dim index is XORed with 8 t = stage_swizzle(row), which spreads a warp's store over all 32 banks and
      // keeps every group of four dims together for the merge's 16-byte loads
      const int sw = t << 3;
      o_sm[h0 * D + (d0 ^ sw)] = st.acc[nt][mt][0];
      o_sm[(h0 + 1) * D + (d0 ^ sw)] = st.acc[nt][mt][1];
      o_sm[h0 * D + ((d0 + kStep) ^ sw)] = st.acc[nt][mt][2];
      o_sm[(h0 + 1) * D + ((d0 + kStep) ^ sw)] = st.acc[nt][mt][3];
    }
  }
}

// Dim-index swizzle of a staged row (see stage_warp_result): rows 2t and 2t+1 of every column tile use 8 t.
__device__ __forceinline__ int stage_swizzle(int row) { return ((row >> 1) & 3) << 3; }

// Merge the NW staged warp results in warp order and write the unit's result: bf16 `out` if the
// sequence is not split, else fp32 partial O (normalised) and its natural-log LSE, per column of the unit.
// o_sm: [NW][o_stride floats], m_sm / l_sm: [NW][NT*8].  `out` is written 8 bytes at a time.
template <int D, int NT, int NW>
__device__ __forceinline__ void merge_and_write(const DecodeParams& p, const Unit& u, const float* o_sm, int o_stride,
                                                const float* m_sm, const float* l_sm, int tid, int nthreads) {
  constexpr int V4 = D / 4;   // a thread merges four consecutive dims of one column: one 16-byte load per warp result
  for (int idx = tid; idx < p.cols * V4; idx += nthreads) {
    const int h = idx / V4;
    const int dim = (idx - h * V4) * 4;
    float m_all = kNegBig;
#pragma unroll
    for (int w = 0; w < NW; ++w) m_all = fmaxf(m_all, m_sm[w * NT * 8 + h]);
    float num[4] = {0.f, 0.f, 0.f, 0.f};
    float den = 0.f;
    const float* src = o_sm + h * D + (dim ^ stage_swizzle(h));
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float mw = m_sm[w * NT * 8 + h];
      const float f = ex2(mw - m_all);   // a warp that saw nothing has l = 0 and O = 0: its factor does not matter
      const float4 o4 = *reinterpret_cast<const float4*>(src + w * o_stride);
      num[0] += f * o4.x;
      num[1] += f * o4.y;
      num[2] += f * o4.z;
      num[3] += f * o4.w;
      den += f * l_sm[w * NT * 8 + h];
    }
    float o[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) o[k] = (den > 0.f) ? num[k] / den * p.v_scale : 0.f;   // den = 0: a query token that sees nothing of this unit
    const int64_t head = col_row(p, u.kvh, h);
    const float lse = (den > 0.f) ? (m_all + lg2(den)) * 0.6931471805599453f : -INFINITY;
    if (u.slot < 0) {
      const __nv_bfloat162 lo = __floats2bfloat162_rn(o[0], o[1]), hi = __floats2bfloat162_rn(o[2], o[3]);
      uint2 packed;
      packed.x = *reinterpret_cast<const uint32_t*>(&lo);
      packed.y = *reinterpret_cast<const uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(p.out + (int64_t(u.b) * p.num_q_heads + head) * D + dim) = packed;
      if (p.lse_out != nullptr && dim == 0) p.lse_out[int64_t(u.b) * p.num_q_heads + head] = lse;
    } else {
      *reinterpret_cast<float4*>(p.partial_o + (int64_t(u.slot) * p.num_q_heads + head) * D + dim) =
          make_float4(o[0], o[1], o[2], o[3]);
      if (dim == 0) p.partial_lse[int64_t(u.slot) * p.num_q_heads + head] = lse;
    }
  }
}

__device__ __forceinline__ void check_planned_length(const DecodeParams& p, const Unit& u, int len_dev) {
  const bool ok = (u.chunk_j == u.n_chunks - 1) ? (u.kv_end == len_dev) : (u.kv_end < len_dev);
  if (!ok) atomicOr(p.error_word, LIBRA_DEV_ERR_SEQ_LEN_MISMATCH);
}

// Output rows of empty sequences are zero; entry e of the plan's empty list (stored after the items).
template <int D>
__device__ __forceinline__ void zero_empty_row(const DecodeParams& p, const int4* entries, int num_items, int e, int tid,
                                               int nthreads) {
  const int64_t row = int64_t(entries[num_items + e].x) * p.num_q_heads * D;
  for (int i = tid; i < p.num_q_heads * D; i += nthreads) p.out[row + i] = __float2bfloat16_rn(0.f);
  if (p.lse_out != nullptr) {
    for (int i = tid; i < p.num_q_heads; i += nthreads) p.lse_out[row / D + i] = -INFINITY;
  }
}

// Programmatic dependent launch, both ends.  launch_dependents: kernels queued behind this one may have
// their blocks scheduled as soon as every block of this grid has got this far (they still wait, inside,
// for this grid to finish).  grid_dependency_wait: this kernel, if it was launched as such a dependent,
// waits here until the grid before it has finished and its writes are visible; a no-op otherwise.
__device__ __forceinline__ void launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

}  // namespace dev

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever completes, with a small
// limit, and must come back with LIBRA_DEV_ERR_WAIT_TIMEOUT recorded instead of hanging.
__global__ void wait_timeout_selftest_kernel(uint32_t* error_word, uint32_t tries) {
  __shared__ uint64_t bar;
  const uint32_t b = dev::smem_u32(&bar);
  if (threadIdx.x == 0) {
    dev::mbar_init(b, 1);
    dev::fence_mbar_init();
  }
  __syncwarp();
  if (!dev::mbar_wait(b, 0, tries) && threadIdx.x == 0) atomicOr(error_word, LIBRA_DEV_ERR_WAIT_TIMEOUT);
}

template <int D, int NW, int STAGES, int EB = 2>   // EB: bytes per cache element
struct DecodeSmem {
  static constexpr int kTileBytes = 16 * D * EB;          // one page of one head: K or V
  static constexpr int kStageBytes = 2 * kTileBytes;      // K then V
  static constexpr int kWarpBytes = STAGES * kStageBytes;
  static constexpr int kRingBytes = NW * kWarpBytes;
  static constexpr int kDynamicBytes = kRingBytes + 1024;  // slack for manual 1024-byte alignment
};

// ------------------------------------------------------------------------------------------------
// One thread block per unit.
// D: head_dim (64 | 128); NT: 8-wide head tiles (1: G <= 8, 2: G <= 16); NW warps; STAGES per warp.
// kLoadsOnly: measurement build of the same kernel - same plan, page walk and copies, but each staged page
// is only touched (one shared-memory word per lane) instead of computed on; `out` gets meaningless values.
// kFp8: the pools hold E4M3 codes; tiles are half as large, the page math is process_page_fp8.
// kAppend: the full build - several query tokens per sequence and the fused append of the newest tokens' rows
// (k_new / v_new).  The plain build knows q_len = 1 and has no append code, which makes its loop leaner.
template <int D, int NT, int NW, int STAGES, bool kLoadsOnly = false, bool kFp8 = false, bool kAppend = false>
// Two shapes are meant to run two blocks per SM and are held to the registers that allows: 6 warps (two column tiles)
// and, over an E4M3 cache, 8 warps x 3 stages with one column tile.
__global__ void __launch_bounds__(NW * 32, (NW == 6 || (kFp8 && NW == 8 && STAGES == 3 && NT == 1)) ? 2 : 1)
decode_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
              const __grid_constant__ DecodeParams p_in, const __grid_constant__ ParamPlan pp) {
  using namespace dev;
  DecodeParams p = p_in;
  if constexpr (!kAppend) {   // one query token, no append: let the compiler fold what depends on them
    p.q_len = 1;
    p.cols = p.group;
    p.hq = p.num_q_heads;
    p.k_new = nullptr;
    p.v_new = nullptr;
  }
  using SM = DecodeSmem<D, NW, STAGES, kFp8 ? 1 : 2>;
  constexpr bool kRows = LIBRA_ROWS_LAYOUT && NT == 2 && !kFp8 && !kLoadsOnly;   // two column tiles of a bf16 cache: columns on the M side
  constexpr int NH = kFp8 ? 1 : D / 64;   // 128-byte column blocks of a row
  static_assert(NT * 8 * D * 4 <= SM::kWarpBytes, "epilogue staging must fit in the warp's ring");

  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t bars[NW * STAGES];
  __shared__ float stat_m[NW][NT * 8];
  __shared__ float stat_l[NW][NT * 8];
  __shared__ int s_last;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* my_ring = ring + warp * SM::kWarpBytes;
  const uint32_t my_ring_u32 = smem_u32(my_ring);
  const uint32_t my_bar0 = smem_u32(&bars[warp * STAGES]);

  // A device-side plan comes with a grid sized for the worst case: most blocks past the first wave have nothing to
  // do.  They find that out first (the counts are only valid once the planning kernel has finished) and leave
  // without setting anything up.
  // The grid's last block zeroes the output rows of all empty sequences (a host plan gives each its own block).
  if (p.dev_counts != nullptr && (blockIdx.x >= sm_count() || blockIdx.x == gridDim.x - 1)) {
    grid_dependency_wait();
    const int n_items = p.dev_counts[plan_layout::kCntItems];
    if (blockIdx.x == gridDim.x - 1) {
      const int n_empty = p.dev_counts[plan_layout::kCntEmpty];
      for (int e = 0; e < n_empty; ++e) zero_empty_row<D>(p, p.entries, n_items, e, threadIdx.x, NW * 32);
      return;
    }
    if (int(blockIdx.x) >= n_items * p.num_kv_heads) return;
  }

  const uint64_t kv_policy = l2_evict_first_policy();
  if (lane == 0) {
    prefetch_tensormap(&map_k);
    prefetch_tensormap(&map_v);
#pragma unroll
    for (int s = 0; s < STAGES; ++s) mbar_init(my_bar0 + 8 * s, 1);
    fence_mbar_init();
  }
  __syncwarp();
  // Up to here nothing was read that an earlier kernel in the stream could have written, so when this
  // launch overlaps the tail of its predecessor the block is resident and set up by the time that ends.
  // With early prefetch (a promise by the caller that the preceding kernel writes neither the block table, the
  // lengths nor any cached row except those of each sequence's newest q_len + 1 tokens) the block goes further
  // before it waits: it walks its block-table row and starts the copies of its first tiles of old tokens.
  // Only a plan that travels in the kernel parameters allows it (a plan in device memory may itself have been
  // written by the preceding kernel).
  const bool early = p.early_prefetch != 0 && p.entries == nullptr && p.dev_counts == nullptr;
  // Ask for the first STAGES tiles per warp of unit `blk` (a block index of this grid) to be brought into L2.
  // (Used at the step boundary only: first-wave blocks warming the units of the NEXT wave as they finish their own
  // gained 1 % on 256 equal units and lost 1 - 2 % on the ragged workloads.)
  // (The host sets l2_warmup only when the plan cannot change under this block's eyes: it travels in the kernel
  // parameters, or it lies in the workspace and an earlier decode launch has already run on it, so that the kernel
  // that wrote it is known to have finished.)
  const bool warm_ok = p.l2_warmup != 0 && blockIdx.x < sm_count();
  auto warm_unit = [&](int blk) {
    const int w_item = blk / p.num_kv_heads;
    const int w_kvh = blk - w_item * p.num_kv_heads;
    const Unit w = decode_unit<NW>((p.entries ? p.entries : pp.e)[w_item], w_kvh, warp);
    if (lane < STAGES && lane < w.n_it) {   // more tiles per warp helped long units and cost the short ones more
      const int tile = w.first_page + warp + lane * NW;
      const int32_t pid = ld_cg_s32(p.block_table + int64_t(w.b) * p.block_table_ld + (tile >> p.tile_shift));
      if (pid >= 0 && int64_t(pid) < p.num_pages) {
        const int tok = (tile & ((1 << p.tile_shift) - 1)) << 4;
        const int c1 = (p.pos_head == 1) ? w_kvh : ((p.pos_page == 1) ? pid : tok);
        const int c2 = (p.pos_head == 2) ? w_kvh : ((p.pos_page == 2) ? pid : tok);
        const int c3 = (p.pos_head == 3) ? w_kvh : ((p.pos_page == 3) ? pid : tok);
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          tma_prefetch_l2_4d(&map_k, h * 64, c1, c2, c3, kv_policy);
          tma_prefetch_l2_4d(&map_v, h * 64, c1, c2, c3, kv_policy);
        }
      }
    }
  };
  if (!early) {
    // Without that promise nothing this block needs may be READ for use before the wait - but it may be asked for.
    // A block of the first wave (resident while the kernel before it drains, DRAM all but idle) looks up the pages
    // of its first tiles and has them brought into L2; ids and data are fetched again, for real, after the wait.  A
    // stale id only warms the wrong lines, a line written later is updated in L2, which is where the copies read.
    if (warm_ok) {
      const int units = p.dev_counts ? p.dev_counts[plan_layout::kCntItems] * p.num_kv_heads : p.num_units;
      if (int(blockIdx.x) < units) warm_unit(int(blockIdx.x));
    }
    grid_dependency_wait();
  }

  // the plan lives in the kernel parameters unless it was too large for them (plain loads: the
  // pointer may address parameter space)
  const int4* entries = p.entries ? p.entries : pp.e;
  int num_items = p.num_items, num_units = p.num_units, num_empty = p.num_empty;
  if (p.dev_counts) {  // planned on the device: the grid is an upper bound, the real counts are here
    num_items = p.dev_counts[plan_layout::kCntItems];
    num_empty = p.dev_counts[plan_layout::kCntEmpty];
    num_units = num_items * p.num_kv_heads;
  }
  if (int(blockIdx.x) >= num_units) {
    if (early) grid_dependency_wait();   // `out` may still be read by the kernel before this one
    if (p.dev_counts == nullptr && int(blockIdx.x) - num_units < num_empty) {
      zero_empty_row<D>(p, entries, num_items, int(blockIdx.x) - num_units, threadIdx.x, NW * 32);
    }
    return;
  }

  // ---- work unit
  const int item_idx = blockIdx.x / p.num_kv_heads;
  const int kvh = blockIdx.x - item_idx * p.num_kv_heads;
  const Unit u = decode_unit<NW>(entries[item_idx], kvh, warp);
  const int n_it = u.n_it;

  // ---- page ids first (the copies wait for them): lane L keeps the id of iteration 32*round + L, one round ahead
  const int32_t* bt_row = p.block_table + int64_t(u.b) * p.block_table_ld;
  const int first_tile = u.first_page + warp;   // tile index within the sequence of this warp's iteration 0
  auto load_ids = [&](int round) -> int32_t {
    const int idx = round * 32 + lane;
    return (idx < n_it) ? __ldg(bt_row + ((first_tile + idx * NW) >> p.tile_shift)) : -1;
  };
  int32_t ids_cur = load_ids(0);
  int32_t ids_nxt = load_ids(1);
  const int len_dev = __ldg(p.seq_lens + u.b);

  // query token i stops seeing the cache q_len - 1 - i tokens before its end; this thread's columns:
  int cut[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      // (two column tiles of a bf16 cache: the columns are rows g and g + 8 of the score tile, kept in cut[0][.])
      const int c = kRows ? (lane >> 2) + 8 * e : nt * 8 + 2 * (lane & 3) + e;
      cut[nt][e] = (p.q_len > 1 && c < p.cols) ? p.q_len - 1 - c / p.group : 0;
    }
  }
  const int common_end = min(u.kv_end, len_dev - (p.q_len - 1));   // tokens below this are seen by every column

  auto issue = [&](int j, int s) {
    if ((j & 31) == 0 && j > 0) {
      ids_cur = ids_nxt;
      ids_nxt = load_ids((j >> 5) + 1);
    }
    const int32_t pid = __shfl_sync(0xffffffffu, ids_cur, j & 31);
    if (lane == 0) {
      if (pid < 0 || int64_t(pid) >= p.num_pages) atomicOr(p.error_word, LIBRA_DEV_ERR_BAD_PAGE_ID);
      const uint32_t bar = my_bar0 + 8 * s;
      const uint32_t kdst = my_ring_u32 + s * SM::kStageBytes;
      const uint32_t vdst = kdst + SM::kTileBytes;
      const int tok = ((first_tile + j * NW) & ((1 << p.tile_shift) - 1)) << 4;   // first token of the tile in its page
      const int c1 = (p.pos_head == 1) ? kvh : ((p.pos_page == 1) ? pid : tok);
      const int c2 = (p.pos_head == 2) ? kvh : ((p.pos_page == 2) ? pid : tok);
      const int c3 = (p.pos_head == 3) ? kvh : ((p.pos_page == 3) ? pid : tok);
      fence_proxy_async();  // earlier generic-proxy accesses to this stage come before the async write
      mbar_expect_tx(bar, SM::kStageBytes);
#pragma unroll
      for (int h = 0; h < NH; ++h) tma_load_4d(kdst + h * 2048, &map_k, bar, h * 64, c1, c2, c3, kv_policy);
#pragma unroll
      for (int h = 0; h < NH; ++h) tma_load_4d(vdst + h * 2048, &map_v, bar, h * 64, c1, c2, c3, kv_policy);
    }
  };

  WarpAcc<D, NT> st;
  st.reset();

  const int pre = n_it < STAGES ? n_it : STAGES;
  int issued = 0;
  if (early) {
    // tokens [0, safe_end) were in the cache before the preceding kernel ran: it may have written this step's
    // newest q_len rows (a cache-write kernel) or the row before them (the fused append of the previous step)
    const int safe_end = len_dev - p.q_len - 1;
    while (issued < pre && u.kv_begin + ((warp + issued * NW) << 4) + 16 <= safe_end) {
      issue(issued, issued);
      ++issued;
    }
    grid_dependency_wait();
  }
  uint32_t qf[NT][D / 16][2];
  if constexpr (kFp8) load_q_frags_fp8<D, NT>(qf, p, u.b, kvh, lane);
  else if constexpr (kRows) load_q_frags_rows<D>(qf, p, u.b, kvh, lane);
  else load_q_frags<D, NT>(qf, p, u.b, kvh, lane);
  for (int j = issued; j < pre; ++j) issue(j, j);
  if (threadIdx.x == 0) check_planned_length(p, u, len_dev);

  bool timed_out = false;
  int s = 0;
  uint32_t parity = 0;
  for (int it = 0; it < n_it; ++it) {
    const uint32_t bar = my_bar0 + 8 * s;
    if (!mbar_wait(bar, parity)) {
      timed_out = true;
      break;
    }
    const uint32_t kt = my_ring_u32 + s * SM::kStageBytes;
    const int tok0 = u.kv_begin + ((warp + it * NW) << 4);
    if constexpr (kLoadsOnly) {
      const uint32_t* words = reinterpret_cast<const uint32_t*>(my_ring + s * SM::kStageBytes);
      st.l[0][0] += float((words[lane * 16] ^ words[SM::kTileBytes / 4 + lane * 16]) & 0xffu);
      st.m[0][0] = 0.f;
    } else {
      if (kAppend && p.k_new != nullptr && tok0 + 16 > len_dev - p.q_len && tok0 < len_dev) {
        // this tile holds some of the sequence's newest q_len tokens: their K and V rows come from k_new / v_new
        // ([batch, q_len, Hkv, D]).  The copy that just landed predates them, so patch the staged tiles (swizzled
        // rows) and write the pools.
        constexpr int EB = kFp8 ? 1 : 2;           // bytes per cache element
        constexpr int kRowChunks = D * EB / 16;    // 16-byte chunks of one row
        const int which = lane / kRowChunks;       // 0: K, 1: V
        const int c16 = lane % kRowChunks;
        const int t_lo = max(tok0, len_dev - p.q_len), t_hi = min(min(tok0 + 16, len_dev), u.kv_end);
        for (int t = t_lo; t < t_hi; ++t) {
          if (which < 2) {
            const int i = t - (len_dev - p.q_len);               // which of the new tokens
            const int64_t page = __ldg(p.block_table + int64_t(u.b) * p.block_table_ld + (t >> (4 + p.tile_shift)));
            const int slot = t & ((16 << p.tile_shift) - 1);     // its slot in that page
            const uint8_t* src = reinterpret_cast<const uint8_t*>(which ? p.v_new : p.k_new) +
                                 ((int64_t(u.b) * p.q_len + i) * p.num_kv_heads + kvh) * (D * EB) + c16 * 16;
            const uint4 row = __ldg(reinterpret_cast<const uint4*>(src));
            uint8_t* tile = my_ring + s * SM::kStageBytes + which * SM::kTileBytes;
            const uint32_t off = kFp8 ? tile_off_fp8<D>(t - tok0, c16) : tile_off(t - tok0, c16);
            *reinterpret_cast<uint4*>(tile + off) = row;
            if (page >= 0 && page < p.num_pages) {
              uint8_t* dst = reinterpret_cast<uint8_t*>(which ? p.v_pool : p.k_pool) +
                             (page * p.stride_page + int64_t(kvh) * p.stride_head + int64_t(slot) * p.stride_token) * EB + c16 * 16;
              *reinterpret_cast<uint4*>(dst) = row;
            }
          }
        }
        fence_proxy_async();  // these generic writes come before the next TMA write into this stage
        __syncwarp();
      }
      if constexpr (kFp8) {
        process_page_fp8<D, NT>(st, qf, kt, kt + SM::kTileBytes, my_ring + s * SM::kStageBytes + SM::kTileBytes,
                             u.kv_end - tok0, p.scale_log2, lane, common_end - tok0, len_dev - tok0, cut);
      } else if constexpr (kRows) {
        process_page_rows<D>(st, qf, kt, kt + SM::kTileBytes, my_ring + s * SM::kStageBytes + SM::kTileBytes,
                             u.kv_end - tok0, p.scale_log2, lane, common_end - tok0, len_dev - tok0, cut);
      } else {
        process_page<D, NT>(st, qf, kt, kt + SM::kTileBytes, my_ring + s * SM::kStageBytes + SM::kTileBytes,
                            u.kv_end - tok0, p.scale_log2, lane, common_end - tok0, len_dev - tok0, cut);
      }
    }
    __syncwarp();  // every lane has consumed the stage before lane 0 refills it
    if (it + STAGES < n_it) issue(it + STAGES, s);
    if (++s == STAGES) {
      s = 0;
      parity ^= 1u;
    }
  }

  // Dependents are let in only now, when this block has streamed its unit: the trigger needs every block of
  // the grid, so the next kernel's first wave becomes resident within the last microseconds of this grid
  // and is released together.  (Triggering at block start lets some of its blocks in much earlier than
  // others; the KV-head blocks of an item then start apart in time, which costs DRAM locality: measured
  // -2 % to -4 % on workloads whose first-wave units are long.)
  launch_dependents();

  if (timed_out) {
    if (lane == 0) atomicOr(p.error_word, LIBRA_DEV_ERR_WAIT_TIMEOUT);
    // give copies that are still in flight one more bounded chance to land before the block exits
    for (int k = 0; k < STAGES; ++k) (void)mbar_wait(my_bar0 + 8 * k, parity);
  }

  // ---- stage (m, l, O) of this warp in its own, now idle, ring; merge the warps; write
  __syncwarp();
  if constexpr (kRows) stage_warp_result_rows<D>(st, reinterpret_cast<float*>(my_ring), stat_m[warp], stat_l[warp], lane);
  else stage_warp_result<D, NT, kFp8>(st, reinterpret_cast<float*>(my_ring), stat_m[warp], stat_l[warp], lane);
  __syncthreads();
  merge_and_write<D, NT, NW>(p, u, reinterpret_cast<const float*>(ring), SM::kWarpBytes / 4, &stat_m[0][0], &stat_l[0][0],
                             threadIdx.x, NW * 32);

  // ---- step C inside this kernel: the block that publishes the last partial of (b, kvh) merges them
  if (u.slot < 0 || !p.fused_combine) return;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    int32_t* cnt = p.counters + int64_t(u.b) * p.num_kv_heads + kvh;
    const int arrived = atomicAdd(cnt, 1);
    s_last = (arrived == u.n_chunks - 1);
    if (s_last) *cnt = 0;  // leave the counter clean for the next launch
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // one warp per column of this KV head, exactly as the combine kernel would do it
  for (int c = warp; c < p.cols; c += NW) {
    combine_row<D>(p.partial_o, p.partial_lse, p.out, u.b, u.slot - u.chunk_j, u.n_chunks, p.num_q_heads,
                   col_row(p, kvh, c), lane, p.lse_out);
  }
}

}  // namespace libra
