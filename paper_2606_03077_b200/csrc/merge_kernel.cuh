// Merge of attention results computed over disjoint parts of the same sequences.
//
// When the tokens of one sequence are spread over several GPUs (not the paper's sharding - its tensor parallelism
// splits the cache by attention head, Section 5.3 - but the remaining way to cut the step), every GPU computes
// out_i and lse_i over its part; after those pairs have been gathered, the result over the whole sequence is
//   M = max_i lse_i ;  w_i = exp(lse_i - M) ;  out = sum_i w_i out_i / sum_i w_i ;  lse = M + ln sum_i w_i
// - the rule of step C, here on the bf16 outputs and float32 LSEs that the decode call returns.
//
// One warp per row; lane i keeps w_i and w_{i+32}; every lane owns D/32 columns; parts are added in index order in
// float32, so the result does not depend on scheduling.  Pure streaming: (n_parts + 1) * D * 2 bytes per row.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace libra {

struct MergeParams {
  const __nv_bfloat16* parts_out;  // [n_parts][rows][D]
  const float* parts_lse;          // [n_parts][rows]
  __nv_bfloat16* out;              // [rows][D]
  float* lse_out;                  // [rows] or null
  int64_t rows;
  int32_t n_parts;                 // 1 .. 64
};

constexpr int kMergeWarps = 8;

template <int D>
__global__ void __launch_bounds__(kMergeWarps * 32) merge_parts_kernel(const MergeParams p) {
  constexpr int V = D / 32;   // columns per lane: 4 or 2
  const int lane = threadIdx.x & 31;
  const int64_t row = int64_t(blockIdx.x) * kMergeWarps + (threadIdx.x >> 5);
  if (row >= p.rows) return;
  const int n = p.n_parts;
  const float l0 = (lane < n) ? __ldg(p.parts_lse + int64_t(lane) * p.rows + row) : -INFINITY;
  const float l1 = (lane + 32 < n) ? __ldg(p.parts_lse + int64_t(lane + 32) * p.rows + row) : -INFINITY;
  float m = fmaxf(l0, l1);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  if (m == -INFINITY) m = 0.f;   // no part holds a token: every weight is 0
  const float w0 = (lane < n) ? expf(l0 - m) : 0.f;
  const float w1 = (lane + 32 < n) ? expf(l1 - m) : 0.f;

  float num[V];
#pragma unroll
  for (int v = 0; v < V; ++v) num[v] = 0.f;
  float den = 0.f;
  const __nv_bfloat16* src = p.parts_out + row * D + lane * V;
  const int64_t stride = p.rows * D;
  for (int i0 = 0; i0 < n; i0 += 4) {
    __nv_bfloat162 x[4][V / 2];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
#pragma unroll
      for (int v = 0; v < V / 2; ++v) x[k][v] = __floats2bfloat162_rn(0.f, 0.f);
      if (i0 + k < n) {
        if constexpr (V == 4) {
          const uint2 raw = __ldg(reinterpret_cast<const uint2*>(src + (i0 + k) * stride));
          x[k][0] = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
          x[k][1] = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
        } else {
          const uint32_t raw = __ldg(reinterpret_cast<const uint32_t*>(src + (i0 + k) * stride));
          x[k][0] = *reinterpret_cast<const __nv_bfloat162*>(&raw);
        }
      }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = i0 + k;
      const float w = __shfl_sync(0xffffffffu, (i < 32) ? w0 : w1, i & 31);   // 0 past n
      den += w;
      if (w != 0.f) {   // a part without tokens may hold anything in its row
#pragma unroll
        for (int v = 0; v < V / 2; ++v) {
          const float2 f = __bfloat1622float2(x[k][v]);
          num[2 * v] += w * f.x;
          num[2 * v + 1] += w * f.y;
        }
      }
    }
  }
  const float inv = (den > 0.f) ? 1.f / den : 0.f;
  if (p.lse_out != nullptr && lane == 0) p.lse_out[row] = (den > 0.f) ? m + logf(den) : -INFINITY;
  __nv_bfloat16* dst = p.out + row * D + lane * V;
#pragma unroll
  for (int v = 0; v < V; v += 2) {
    *reinterpret_cast<__nv_bfloat162*>(dst + v) = __floats2bfloat162_rn(num[v] * inv, num[v + 1] * inv);
  }
}

}  // namespace libra
