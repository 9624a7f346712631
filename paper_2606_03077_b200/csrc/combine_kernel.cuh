// Combine kernel (step C): log-sum-exp merge of the partial results of split sequences.
//
// For sequence b, head h with n partials (O_i normalised, LSE_i natural log):
//   M = max_i LSE_i ;  w_i = exp(LSE_i - M) ;  out = sum_i w_i O_i / sum_i w_i   -> bf16
// Partials are summed in chunk order, so the result does not depend on scheduling.  An entry with
// n == 0 is an empty sequence: its output row is zero.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "plan_layout.hpp"

namespace libra {

struct CombineParams {
  const int32_t* plan;
  const float* partial_o;    // [slot][Hq][D]
  const float* partial_lse;  // [slot][Hq]
  const int32_t* seq_lens;
  __nv_bfloat16* out;        // [B][Hq][D]
  uint32_t* error_word;
  int32_t num_q_heads;
  int32_t head_dim;
};

// grid = (fix-up entries, query heads), block = head_dim / 2 threads, two output dims per thread
__global__ void combine_kernel(const CombineParams p) {
  const int32_t* fix = p.plan + __ldg(p.plan + plan_layout::kFixOff) + blockIdx.x * plan_layout::kFixInts;
  const int b = __ldg(fix + 0);
  const int first = __ldg(fix + 1);
  const int n = __ldg(fix + 2);
  const int h = blockIdx.y;
  const int Hq = p.num_q_heads;
  const int D = p.head_dim;
  if (threadIdx.x == 0 && h == 0 && __ldg(fix + 3) != __ldg(p.seq_lens + b)) {
    atomicOr(p.error_word, LIBRA_DEV_ERR_SEQ_LEN_MISMATCH);
  }
  float m = -INFINITY;
  for (int i = 0; i < n; ++i) m = fmaxf(m, __ldg(p.partial_lse + int64_t(first + i) * Hq + h));
  float2 num = make_float2(0.f, 0.f);
  float den = 0.f;
  for (int i = 0; i < n; ++i) {
    const int64_t row = int64_t(first + i) * Hq + h;
    const float w = __expf(__ldg(p.partial_lse + row) - m);
    const float2 o = __ldg(reinterpret_cast<const float2*>(p.partial_o + row * D) + threadIdx.x);
    num.x += w * o.x;
    num.y += w * o.y;
    den += w;
  }
  const float inv = (n > 0) ? 1.f / den : 0.f;
  __nv_bfloat162 r = __floats2bfloat162_rn(num.x * inv, num.y * inv);
  reinterpret_cast<__nv_bfloat162*>(p.out + (int64_t(b) * Hq + h) * D)[threadIdx.x] = r;
}

}  // namespace libra
