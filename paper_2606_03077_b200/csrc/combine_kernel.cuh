// Combine kernel (step C): log-sum-exp merge of the partial results of split sequences.
//
// For sequence b, head h with n partials (O_i normalised, LSE_i natural log):
//   M = max_i LSE_i ;  w_i = exp(LSE_i - M) ;  out = sum_i w_i O_i / sum_i w_i   -> bf16
// Partials are summed in chunk order, so the result does not depend on scheduling.
//
// One warp per (sequence, head) row: lane i keeps w_i and w_{i+32}; every lane owns D/32 output
// columns and walks the n partial rows with eight independent loads in flight.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "plan_layout.hpp"

namespace libra {

struct CombineParams {
  const int4* entries;       // merges {b, first_slot, n, planned_len} in device memory, or null: in `pf`
  const int32_t* dev_counts; // device-side plan: the number of merges is read from here (null = host plan)
  const float* partial_o;    // [slot][Hq][D]
  const float* partial_lse;  // [slot][Hq]
  const int32_t* seq_lens;
  __nv_bfloat16* out;        // [B][Hq][D]
  float* lse_out;            // [B][Hq] natural-log sum of exponentials of each row, or null
  uint32_t* error_word;
  int32_t num_q_heads;
};

constexpr int kCombineWarps = 4;

// One warp merges the n (<= 64) partial results of one (sequence, head) row and writes the bf16 row.
// Shared by the combine kernel and by the decode kernel's in-kernel merge, so both give the same bits.
// Loads bypass L1 (the partials were written by other SMs, possibly during this very launch).
// lse_out (nullable): the row's final LSE = M + ln(sum_i w_i) goes to lse_out[b * Hq + h].
template <int D>
__device__ __forceinline__ void combine_row(const float* partial_o, const float* partial_lse, __nv_bfloat16* out, int b,
                                            int first, int n, int Hq, int h, int lane, float* lse_out = nullptr) {
  constexpr int V = D / 32;  // columns per lane: 4 (float4) or 2 (float2)
  const float* lse = partial_lse + int64_t(first) * Hq + h;
  const float l0 = (lane < n) ? __ldcg(lse + int64_t(lane) * Hq) : -INFINITY;
  const float l1 = (lane + 32 < n) ? __ldcg(lse + int64_t(lane + 32) * Hq) : -INFINITY;
  float m = fmaxf(l0, l1);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  if (m == -INFINITY) m = 0.f;  // no partial holds anything (a query token that sees no cached token): all weights 0
  const float w0 = (lane < n) ? __expf(l0 - m) : 0.f;
  const float w1 = (lane + 32 < n) ? __expf(l1 - m) : 0.f;

  float num[V];
#pragma unroll
  for (int v = 0; v < V; ++v) num[v] = 0.f;
  float den = 0.f;
  const float* po = partial_o + (int64_t(first) * Hq + h) * D + lane * V;
  const int64_t stride = int64_t(Hq) * D;
  for (int i0 = 0; i0 < n; i0 += 8) {
    float o[8][V];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if (i0 + k < n) {
        if constexpr (V == 4) {
          const float4 x = __ldcg(reinterpret_cast<const float4*>(po + (i0 + k) * stride));
          o[k][0] = x.x; o[k][1] = x.y; o[k][2] = x.z; o[k][3] = x.w;
        } else {
          const float2 x = __ldcg(reinterpret_cast<const float2*>(po + (i0 + k) * stride));
          o[k][0] = x.x; o[k][1] = x.y;
        }
      } else {
#pragma unroll
        for (int v = 0; v < V; ++v) o[k][v] = 0.f;
      }
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int i = i0 + k;
      const float w = __shfl_sync(0xffffffffu, (i < 32) ? w0 : w1, i & 31);  // 0 past n
      den += w;
#pragma unroll
      for (int v = 0; v < V; ++v) num[v] += w * o[k][v];
    }
  }
  const float inv = (den > 0.f) ? 1.f / den : 0.f;
  if (lse_out != nullptr && lane == 0) lse_out[int64_t(b) * Hq + h] = (den > 0.f) ? m + __logf(den) : -INFINITY;
  __nv_bfloat16* dst = out + (int64_t(b) * Hq + h) * D + lane * V;
#pragma unroll
  for (int v = 0; v < V; v += 2) {
    *reinterpret_cast<__nv_bfloat162*>(dst + v) = __floats2bfloat162_rn(num[v] * inv, num[v + 1] * inv);
  }
}

// grid = (fix-up entries, ceil(Hq / kCombineWarps)), block = kCombineWarps warps
template <int D>
__global__ void __launch_bounds__(kCombineWarps * 32)
combine_kernel(const __grid_constant__ CombineParams p, const __grid_constant__ ParamFix pf) {
  // Launched as a programmatic dependent of the decode kernel: wait until that grid has finished and its
  // partial results (and a device-side plan's counts) are visible.  EVERY thread waits, also those that have
  // nothing to do: a grid that completes without waiting would let whatever follows it in the stream start
  // while the decode kernel is still running.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int lane = threadIdx.x & 31;
  const int h = blockIdx.y * kCombineWarps + (threadIdx.x >> 5);
  const int Hq = p.num_q_heads;
  if (h >= Hq) return;
  if (p.dev_counts && int(blockIdx.x) >= p.dev_counts[plan_layout::kCntCombine]) return;  // grid is an upper bound
  const int4 fix = (p.entries ? p.entries : pf.e)[blockIdx.x];  // plain load: may address parameter space
  if (lane == 0 && h == 0 && fix.w != __ldg(p.seq_lens + fix.x)) {
    atomicOr(p.error_word, LIBRA_DEV_ERR_SEQ_LEN_MISMATCH);
  }
  combine_row<D>(p.partial_o, p.partial_lse, p.out, fix.x, fix.y, fix.z, Hq, h, lane, p.lse_out);
}

}  // namespace libra
