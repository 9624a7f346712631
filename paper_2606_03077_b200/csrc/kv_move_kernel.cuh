// KV gather / scatter kernels: the data movement of a request's migration between rollout buckets.
//
// The paper moves a paused request's KV cache in three steps (Section 5.3): offload to pinned host
// memory, reshard along the attention-head dimension to the target bucket's tensor-parallel degree
// (split a source partition into TP_tgt / TP_src shards, or concatenate TP_src / TP_tgt of them), and
// reload on the target GPUs.  Here the reshard is not a pass of its own: a head range is an argument of
// both kernels, so a gather already produces the target shard and a scatter already lands it at the
// right head offset.
//
//   gather : pages of the listed sequences, heads [head_begin, head_begin + head_count) of the pool
//            -> dense rows  dst[(token_offset[b] + t) * head_count + (h - head_begin)][0 .. D)
//   scatter: the inverse, into the pages the (new) block table names, at heads
//            [head_begin, head_begin + head_count) of the destination pool
//
// `dense` may be device memory or pinned host memory mapped into the device's address space.
// Pure copies: bound by memory bandwidth (read + write = 2 x the bytes moved), no arithmetic.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace libra {

struct KvMoveParams {
  __nv_bfloat16* k_pool;        // paged pools (read by gather, written by scatter)
  __nv_bfloat16* v_pool;
  __nv_bfloat16* k_dense;       // dense shard buffers (written by gather, read by scatter)
  __nv_bfloat16* v_dense;
  const int32_t* block_table;   // [batch][ld]
  const int32_t* seq_lens;      // [batch]
  const int64_t* token_offsets; // [batch]: first dense row (in tokens) of each sequence
  int64_t stride_page, stride_head, stride_token;  // pool strides in elements
  int64_t num_pages;
  int32_t block_table_ld;
  int32_t head_begin, head_count;
  int32_t page_size;            // tokens per page (16, 32 or 64)
  uint32_t* error_word;
};

constexpr int kMovePagesPerBlock = 4;
constexpr int kMoveThreads = 256;

// grid = (ceil(max pages per sequence / kMovePagesPerBlock), batch); block = kMoveThreads.
// One 16-byte vector per thread per step; a (page, head) tile is page_size tokens x D elements.
template <int D, bool kGather>
__global__ void __launch_bounds__(kMoveThreads) kv_move_kernel(const KvMoveParams p) {
  constexpr int VEC = 8;                    // bf16 per 16-byte vector
  constexpr int VPR = D / VEC;              // vectors per token row of one head
  const int b = blockIdx.y;
  const int len = __ldg(p.seq_lens + b);
  const int P = p.page_size;
  const int n_pages = (len + P - 1) / P;
  const int page0 = blockIdx.x * kMovePagesPerBlock;
  if (page0 >= n_pages) return;
  const int page1 = min(n_pages, page0 + kMovePagesPerBlock);
  const int64_t row0 = __ldg(p.token_offsets + b);
  const int vec_per_page = P * p.head_count * VPR;    // token-major inside the page: (token, head, vec)

  for (int pg = page0; pg < page1; ++pg) {
    const int64_t pid = __ldg(p.block_table + int64_t(b) * p.block_table_ld + pg);
    if (pid < 0 || pid >= p.num_pages) {
      if (threadIdx.x == 0) atomicOr(p.error_word, LIBRA_DEV_ERR_BAD_PAGE_ID);
      continue;
    }
    const int valid = min(P, len - pg * P);
    for (int i = threadIdx.x; i < vec_per_page; i += kMoveThreads) {
      const int vec = i % VPR;
      const int head = (i / VPR) % p.head_count;
      const int tok = i / (VPR * p.head_count);
      if (tok >= valid) continue;
      const int64_t pool_off = pid * p.stride_page + int64_t(p.head_begin + head) * p.stride_head +
                               int64_t(tok) * p.stride_token + vec * VEC;
      const int64_t dense_off = ((row0 + int64_t(pg) * P + tok) * p.head_count + head) * D + vec * VEC;
      if (kGather) {
        *reinterpret_cast<uint4*>(p.k_dense + dense_off) = __ldg(reinterpret_cast<const uint4*>(p.k_pool + pool_off));
        *reinterpret_cast<uint4*>(p.v_dense + dense_off) = __ldg(reinterpret_cast<const uint4*>(p.v_pool + pool_off));
      } else {
        *reinterpret_cast<uint4*>(p.k_pool + pool_off) = __ldg(reinterpret_cast<const uint4*>(p.k_dense + dense_off));
        *reinterpret_cast<uint4*>(p.v_pool + pool_off) = __ldg(reinterpret_cast<const uint4*>(p.v_dense + dense_off));
      }
    }
  }
}

}  // namespace libra
