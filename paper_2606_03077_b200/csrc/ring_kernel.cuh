// Data plane of the inter-replica ring all-reduce: one step on one GPU.
//
// In the paper the CPU owns membership, transport and flow control of the gradient exchange between replicas and
// the GPU only copies and reduces chunks of a ring ReduceScatter + AllGather; its kernel busy-polls a host-pinned
// "data has arrived" flag with a software timeout instead of blocking, and is written to get by on 2 SMs so that
// it does not take SMs from the computation it overlaps with (Section 6, "Decoupled communication domains"; appendix
// "Decoupled Communication Domain").  This is that step:
//
//   wait, bounded, until *ready >= expected          (flag in host-pinned or device memory, written by the host
//                                                      or by whoever delivered the chunk)
//   REDUCE : dst[i] = own[i] + received[i]            one ReduceScatter step   (float32, or bfloat16 summed in float32
//   COPY   : dst[i] = received[i]                     one AllGather step        and rounded to nearest even)
//
// A few blocks (2 by default) of 512 threads; every thread keeps kRingUnroll 16-byte loads of each operand in flight,
// which is what lets so few SMs stream at a useful rate.  If the wait runs out nothing but the status word is
// written; the context stays usable.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace libra {

constexpr int kRingThreads = 512;
constexpr int kRingUnroll = 8;

struct RingStepParams {
  void* dst;
  const void* own;            // null for COPY
  const void* received;
  size_t n16;                 // 16-byte vectors (whole vectors only; the caller pads chunks to 16 bytes)
  const uint32_t* status;     // device word written by ring_wait_kernel: 0 = go, 1 = the wait ran out
  int32_t bf16;               // element type: 0 float32, 1 bfloat16
};

namespace dev {

__device__ __forceinline__ uint32_t ld_flag(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.relaxed.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// A streaming 16-byte load on the coherent path (not `.nc`): `dst` may be `own` (in-place ReduceScatter), and the
// read-only path is defined only for memory that nothing writes while the kernel runs.
__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p)
               : "memory");
  return v;
}
__device__ __forceinline__ uint32_t add_bf16x2(uint32_t a, uint32_t b) {
  const float lo = __uint_as_float(a << 16) + __uint_as_float(b << 16);
  const float hi = __uint_as_float(a & 0xffff0000u) + __uint_as_float(b & 0xffff0000u);
  const __nv_bfloat162 r = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&r);
}
__device__ __forceinline__ uint4 add16(uint4 a, uint4 b, bool bf16) {
  uint4 r;
  if (bf16) {
    r.x = add_bf16x2(a.x, b.x); r.y = add_bf16x2(a.y, b.y); r.z = add_bf16x2(a.z, b.z); r.w = add_bf16x2(a.w, b.w);
  } else {
    r.x = __float_as_uint(__uint_as_float(a.x) + __uint_as_float(b.x));
    r.y = __float_as_uint(__uint_as_float(a.y) + __uint_as_float(b.y));
    r.z = __float_as_uint(__uint_as_float(a.z) + __uint_as_float(b.z));
    r.w = __float_as_uint(__uint_as_float(a.w) + __uint_as_float(b.w));
  }
  return r;
}

}  // namespace dev

// The wait is a kernel of its own, one thread: it polls the flag, bounded by the clock (timeout_us) and by an
// iteration count, and writes the verdict to the status word.  The copy / reduce kernel behind it in the stream
// reads the verdict, so all of its blocks agree on it (blocks polling on their own could disagree when the flag
// arrives at the deadline), and no SM is held while waiting.
__global__ void ring_wait_kernel(const uint32_t* ready, uint32_t expected, uint32_t timeout_us, uint32_t* status) {
  using namespace dev;
  if (threadIdx.x != 0) return;
  const uint64_t t0 = global_timer_ns();
  const uint64_t limit = uint64_t(timeout_us) * 1000ull;
  uint32_t verdict = 1u;
  for (uint32_t it = 0; it < (1u << 26); ++it) {
    if (ld_flag(ready) >= expected) {
      verdict = 0u;
      break;
    }
    if (global_timer_ns() - t0 > limit) break;
    __nanosleep(200);
  }
  __threadfence_system();   // the chunk was written before the flag: what follows in the stream reads it after the flag
  *status = verdict;
}

// grid = a few blocks (2 by default), block = kRingThreads; runs behind ring_wait_kernel in the same stream
__global__ void __launch_bounds__(kRingThreads) ring_step_kernel(const RingStepParams p) {
  using namespace dev;
  if (*p.status != 0u) return;   // the wait ran out: write nothing

  const uint4* recv = static_cast<const uint4*>(p.received);
  const uint4* own = static_cast<const uint4*>(p.own);
  uint4* dst = static_cast<uint4*>(p.dst);
  const bool bf16 = p.bf16 != 0;
  const size_t stride = size_t(gridDim.x) * kRingThreads;
  size_t i = size_t(blockIdx.x) * kRingThreads + threadIdx.x;
  for (; i + (kRingUnroll - 1) * stride < p.n16; i += kRingUnroll * stride) {
    uint4 a[kRingUnroll], b[kRingUnroll];
#pragma unroll
    for (int k = 0; k < kRingUnroll; ++k) a[k] = ld_stream16(recv + i + k * stride);
    if (own) {
#pragma unroll
      for (int k = 0; k < kRingUnroll; ++k) b[k] = ld_stream16(own + i + k * stride);
#pragma unroll
      for (int k = 0; k < kRingUnroll; ++k) a[k] = add16(b[k], a[k], bf16);
    }
#pragma unroll
    for (int k = 0; k < kRingUnroll; ++k) dst[i + k * stride] = a[k];
  }
  for (; i < p.n16; i += stride) {
    uint4 a = ld_stream16(recv + i);
    if (own) a = add16(ld_stream16(own + i), a, bf16);
    dst[i] = a;
  }
}

}  // namespace libra
