// Device-side planner (step P on the GPU): the same length-bucketed rule as planner.cpp, computed by
// one thread block from the device copy of the sequence lengths, so that a whole decode step (plan,
// decode, combine) can be enqueued - or captured in a CUDA graph - without the host ever seeing the
// lengths.  The paper re-plans as the length distribution drifts (Section 4.3: the planner is re-run
// every K iterations; Section 2.2: lengths grow during training); here that means every step.
//
//   C       = max(min_chunk, au(cd(heads * T, slots), chunk_align))          T = sum of lengths
//   s_b     = min(p2(cd(L_b, C)), max_splits)      chunk_b = au(cd(L_b, s_b), chunk_align)
//   n_b     = cd(L_b, chunk_b)                     items sorted by (length desc, b asc, j asc)
//   a plan of fewer than one and a half waves of long blocks is made again for twice as many slots (plan_layout.hpp)
//
// Integer arithmetic only; the result must equal the host planner's bit for bit.  Limits: batch and
// work items <= kDevPlanMax each (one block of up to 1024 threads, four elements per thread; the block is sized to the
// batch, because its barriers and scans are what its time is made of); beyond that, or when a length
// exceeds what a block-table row can describe, the kernel writes an empty plan and sets
// LIBRA_DEV_ERR_PLAN_OVERFLOW.  Negative lengths count as empty sequences.
#pragma once
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>

#include "plan_layout.hpp"

namespace libra {

constexpr int kDevPlanThreads = 1024;   // the most threads one planning block has
constexpr int kDevPlanPerThread = 4;
constexpr int kDevPlanMax = kDevPlanThreads * kDevPlanPerThread;
// Items up to which the quadratic ranking loop is used; above, a radix sort in shared memory (a bitonic sort if a
// work unit has 2^16 tokens or more).  Measured on a B200, one planning kernel in a chain of them, of which the
// ordering step: 64 items 4.3 us (0.3), 256 items 6.7 (2.4), 384 items 9.8 (5.1) with the loop, which takes 44 us at 1024
// items and about 150 us at 2048; with the radix sort 512 items 8.5 us (3.4), 1024 items 11.7 (4.9), 2048 items 14.9
// (6.3), 4096 items 21.3 (9.7); the bitonic sort takes 6.8 / 11.7 / 21.8 / 42.9 us at those four sizes.
constexpr int kDevPlanRankLoopMax = 256;
constexpr int kDevPlanArrays = 10;      // shared-memory arrays of kDevPlanPerThread * blockDim.x ints each
constexpr int kDevPlanRadixMaxLen = 1 << 16;   // the radix sort packs (length, index) into one word: lengths below this

struct PlanKernelParams {
  const int32_t* seq_lens;   // device, [batch]
  int32_t batch;
  int32_t heads;             // work units per item (KV heads)
  int64_t slots;             // n_sm * ctas_per_sm * items_per_slot
  int32_t chunk_align, min_chunk, max_splits;
  int64_t wave_slots;        // n_sm * ctas_per_sm: thread blocks of one wave
  int32_t refine;            // 1: a coarse plan of long blocks is made again for twice as many slots
  int32_t max_items;         // capacity of `entries` for work items
  int32_t max_len;           // longest sequence the block table can describe
  int32_t* counts;           // [plan_layout::kCountInts]: num_items, num_combine, num_empty, chunk_target, overflow
  int32_t* per_seq;          // [4][batch]: bucket, num_splits, chunk_len, item_offset
  int4* entries;             // work items, then one entry per empty sequence
  int4* fixes;               // merges for the combine kernel
  uint32_t* error_word;
};

// Threads of the planning block for a batch and an item bound: every thread owns up to kDevPlanPerThread elements
// of each array; a small batch gets a small block (its barriers and scans are what the kernel's time is made of).
inline int plan_kernel_threads(int64_t batch, int64_t item_bound) {
  // one element per thread where that fits in a block (the ranking step is quadratic in the items), never fewer
  // threads than the arrays need
  const int64_t n = std::max<int64_t>(std::max(batch, item_bound), 1);
  return int(std::min<int64_t>(kDevPlanThreads, std::max<int64_t>(128, (n + 31) / 32 * 32)));
}
inline size_t plan_kernel_smem_bytes(int threads) {
  return size_t(kDevPlanArrays) * kDevPlanPerThread * threads * sizeof(int);
}

namespace dev {

// Exclusive scan of `n` ints in shared memory (n <= kDevPlanPerThread * blockDim.x), in place; returns the total.
// `warp_tot` is scratch for 33 ints.  All threads of the block call it.
__device__ __forceinline__ int block_exclusive_scan(int* data, int n, int* warp_tot) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;
  int v[kDevPlanPerThread];
  int sum = 0;
#pragma unroll
  for (int k = 0; k < kDevPlanPerThread; ++k) {
    const int i = tid * kDevPlanPerThread + k;
    v[k] = (i < n) ? data[i] : 0;
    sum += v[k];
  }
  int incl = sum;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = (lane < n_warps) ? warp_tot[lane] : 0;
    int wi = w;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, wi, off);
      if (lane >= off) wi += t;
    }
    warp_tot[lane] = wi - w;  // exclusive prefix of the warp totals
    if (lane == 31) warp_tot[32] = wi;
  }
  __syncthreads();
  int run = warp_tot[warp] + incl - sum;
#pragma unroll
  for (int k = 0; k < kDevPlanPerThread; ++k) {
    const int i = tid * kDevPlanPerThread + k;
    if (i < n) data[i] = run;
    run += v[k];
  }
  const int total = warp_tot[32];
  __syncthreads();
  return total;
}

// ceil(a / b) for 0 <= a < 2^31 and b >= 1 (b may exceed 32 bits: then the quotient is 0 or 1)
__device__ __forceinline__ int ceil_div_len(int a, long long b) {
  if (b > 0x7fffffffll) return a > 0 ? 1 : 0;
  const unsigned ub = unsigned(b);
  return int((unsigned(a) + ub - 1u) / ub);
}

}  // namespace dev

// grid = 1 block of plan_kernel_threads(batch, item bound) threads; dynamic shared memory = plan_kernel_smem_bytes(threads)
__global__ void __launch_bounds__(kDevPlanThreads) plan_kernel(const PlanKernelParams p) {
  extern __shared__ int sm[];
  const int cap = kDevPlanPerThread * int(blockDim.x);
  int* len_s = sm;                // [batch] lengths (negative ones taken as 0)
  int* nsplit = sm + cap;         // [batch]
  int* chunk = sm + 2 * cap;      // [batch]
  int* offs = sm + 3 * cap;       // [batch] exclusive scan of nsplit
  int* aux = sm + 4 * cap;        // [batch] flags / their scans
  int* it_len = sm + 5 * cap;     // [items]
  int* it_b = sm + 6 * cap;       // [items]
  int* it_j = sm + 7 * cap;       // [items]
  int* hist = sm + 8 * cap;       // [warps][256] digit counts of the radix sort (two arrays: 8 ints per thread)
  __shared__ int digit_tot[256];
  __shared__ int warp_tot[33];
  __shared__ long long warp_sum[32];

  const int tid = threadIdx.x, nthr = blockDim.x;
  const int B = p.batch;
  namespace L = plan_layout;

  // Programmatic dependent launch, both ends.  This kernel may be launched as a dependent of whatever precedes it in
  // the stream (the previous step's decode kernel, or the kernel that wrote the lengths): it waits here until that
  // grid has finished - the lengths it reads and the plan region it overwrites are then free.  Right after, it lets
  // the kernel behind it (the decode kernel of this step) have its blocks scheduled: they set themselves up on the
  // other SMs while this one block plans, and wait, inside, for this grid to finish before they read the plan.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  auto refuse = [&](int base_out) {
    if (tid == 0) {
      p.counts[L::kCntItems] = 0; p.counts[L::kCntCombine] = 0; p.counts[L::kCntEmpty] = 0;
      p.counts[L::kCntChunkTarget] = base_out; p.counts[L::kCntOverflow] = 1;
      atomicOr(p.error_word, LIBRA_DEV_ERR_PLAN_OVERFLOW);
    }
  };
  if (B > cap) {   // more sequences than this block was sized for
    refuse(0);
    return;
  }

  // ---- the lengths, once, into shared memory; T = their sum
  long long part = 0;
  int too_long = 0;
  for (int b = tid; b < B; b += nthr) {
    const int len = p.seq_lens[b];
    too_long |= (len > p.max_len) ? 1 : 0;
    len_s[b] = max(len, 0);
    part += max(len, 0);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
  if ((tid & 31) == 0) warp_sum[tid >> 5] = part;
  if (__syncthreads_or(too_long)) {  // a length the block table cannot hold: refuse the whole batch
    refuse(0);
    return;
  }
  long long T = 0;
  for (int w = 0; w < (nthr >> 5); ++w) T += warp_sum[w];
  const long long A = p.chunk_align;
  long long base = (p.heads * T + p.slots - 1) / p.slots;
  base = (base + A - 1) / A * A;
  if (base < p.min_chunk) base = p.min_chunk;

  // ---- per sequence: degree, chunk length, chunk count; twice if the first plan is coarse
  int n_items = 0;
  for (int pass = 0; pass < 2; ++pass) {
    for (int b = tid; b < B; b += nthr) {
      const int len = len_s[b];
      int bucket = -1, n = 0, c = 0;
      if (len > 0) {
        const int want = dev::ceil_div_len(len, base);
        int deg = 1;
        bucket = 0;
        while (deg < want) {
          deg <<= 1;
          ++bucket;
        }
        if (base < plan_layout::kSmallBaseTokens && deg > 1 &&
            (long long)len * plan_layout::kGeoMeanDen < (long long)(deg / 2) * base * plan_layout::kGeoMeanNum) {
          deg >>= 1;   // short chunks: the nearer power of two
          --bucket;
        }
        while (deg > p.max_splits) {
          deg >>= 1;
          --bucket;
        }
        const unsigned a = unsigned(A);
        const unsigned per = (unsigned(len) + unsigned(deg) - 1u) >> bucket;   // ceil(len / deg), deg = 2^bucket
        c = int((per + a - 1u) / a * a);
        n = int((unsigned(len) + unsigned(c) - 1u) / unsigned(c));
      }
      nsplit[b] = n;
      chunk[b] = c;
      offs[b] = n;
      p.per_seq[b] = bucket;
    }
    __syncthreads();
    n_items = dev::block_exclusive_scan(offs, B, warp_tot);
    // fewer than one and a half waves of long blocks: once more, for twice as many slots (the same for every thread)
    if (pass == 1 || !p.refine || base < plan_layout::kRefineMinBaseTokens ||
        (long long)plan_layout::kRefineWavesDen * p.heads * n_items >= plan_layout::kRefineWavesNum * p.wave_slots) {
      break;
    }
    base = (p.heads * T + 2 * p.slots - 1) / (2 * p.slots);
    base = (base + A - 1) / A * A;
    if (base < p.min_chunk) base = p.min_chunk;
  }
  for (int b = tid; b < B; b += nthr) {
    p.per_seq[B + b] = nsplit[b];
    p.per_seq[2 * B + b] = chunk[b];
    p.per_seq[3 * B + b] = offs[b];
  }

  if (n_items > cap || n_items > p.max_items) {
    refuse(int(base));
    return;
  }

  // ---- merges (n_b > 1) and empty sequences, each in batch order: one scan counts both (16 bits each)
  for (int b = tid; b < B; b += nthr) aux[b] = (nsplit[b] > 1 ? 1 : 0) | (nsplit[b] == 0 ? (1 << 16) : 0);
  __syncthreads();
  const int both = dev::block_exclusive_scan(aux, B, warp_tot);
  const int n_combine = both & 0xffff, n_empty = both >> 16;
  for (int b = tid; b < B; b += nthr) {
    if (nsplit[b] > 1) p.fixes[aux[b] & 0xffff] = make_int4(b, offs[b], nsplit[b], len_s[b]);
    if (nsplit[b] == 0) p.entries[n_items + (aux[b] >> 16)] = make_int4(b, 0, 0, 0);
  }

  // ---- items in (b, j) order (the list is padded to a multiple of four with lengths that rank after everything)
  if (tid < 4 && (n_items & ~3) + tid >= n_items && (n_items & ~3) + tid < cap) it_len[(n_items & ~3) + tid] = -1;
  int wide = 0;
  for (int b = tid; b < B; b += nthr) {
    const int len = len_s[b];
    wide |= (chunk[b] >= kDevPlanRadixMaxLen) ? 1 : 0;
    for (int j = 0; j < nsplit[b]; ++j) {
      const int i = offs[b] + j;
      const int lo = j * chunk[b];
      const int hi = min(len, lo + chunk[b]);
      it_len[i] = hi - lo;
      it_b[i] = b;
      it_j[i] = j;
    }
  }
  wide = __syncthreads_or(wide);

  auto emit = [&](int rank, int i) {
    const int b = it_b[i], j = it_j[i];
    const int lo = j * chunk[b];
    const int hi = min(len_s[b], lo + chunk[b]);
    p.entries[rank] = make_int4(b | (j << L::kChunkShift) | (nsplit[b] << L::kCountShift), lo, hi,
                                (nsplit[b] > 1) ? offs[b] + j : -1);
  };

  auto finish = [&]() {
    if (tid == 0) {
      p.counts[L::kCntItems] = n_items;
      p.counts[L::kCntCombine] = n_combine;
      p.counts[L::kCntEmpty] = n_empty;
      p.counts[L::kCntChunkTarget] = int(base);
      p.counts[L::kCntOverflow] = 0;
    }
  };

  if (n_items > kDevPlanRankLoopMax && !wide) {
    // ---- many items, lengths below 2^16: a stable radix sort, two passes of 8 bits, of the words
    // (0xffff - length) << 16 | index.  Ascending and stable, so longest first with ties in index order, which is
    // the (b, j) order.  Warp w owns the items [w * per, (w + 1) * per), 32 at a time: within a warp the items of one
    // digit are ranked by warp votes and a per-warp counter, across warps by a scan of the counters.
    const int lane = tid & 31, warp = tid >> 5, n_warps = nthr >> 5;
    const int per = ((n_items + n_warps - 1) / n_warps + 31) & ~31;      // <= 128: n_items <= cap = 128 * n_warps
    unsigned* src = reinterpret_cast<unsigned*>(it_len);
    unsigned* dst = reinterpret_cast<unsigned*>(aux);                     // the flags in aux were last read before the barrier above
    for (int i = tid; i < n_items; i += nthr) src[i] = (unsigned(0xffff - it_len[i]) << 16) | unsigned(i);
    for (int shift = 16; shift < 32; shift += 8) {
      for (int i = tid; i < n_warps * 64; i += nthr) reinterpret_cast<int4*>(hist)[i] = make_int4(0, 0, 0, 0);
      __syncthreads();
      int loc[4], dig[4];
      unsigned word[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        dig[e] = 256;
        if (e * 32 >= per) continue;                                       // the same for the whole warp
        const int i = warp * per + e * 32 + lane;
        const bool live = i < n_items;
        word[e] = live ? src[i] : 0u;
        const unsigned d = (word[e] >> shift) & 255u;
        // the lanes that hold the same digit: eight votes, one per bit (the hardware's match instruction takes a
        // round per distinct value, up to 32 of them here)
        unsigned grp = __ballot_sync(0xffffffffu, live);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const unsigned vote = __ballot_sync(0xffffffffu, (d >> k) & 1u);
          grp &= ((d >> k) & 1u) ? vote : ~vote;
        }
        int first = 0;
        if (live) {
          dig[e] = int(d);
          const int leader = __ffs(grp) - 1;
          if (lane == leader) {
            first = hist[warp * 256 + d];
            hist[warp * 256 + d] = first + __popc(grp);
          }
          // every lane of a group reads its leader's value; groups are disjoint, so one shuffle serves them all
        }
        const int src_lane = live ? __ffs(grp) - 1 : lane;
        loc[e] = __shfl_sync(0xffffffffu, first, src_lane) + __popc(grp & ((1u << lane) - 1u));
        __syncwarp();                                                      // the counter's new value, before the next 32 items
      }
      __syncthreads();
      for (int d = tid; d < 256; d += nthr) {   // per digit: the warps' counts become their exclusive prefix, the total goes to digit_tot
        int run = 0;
        for (int w0 = 0; w0 < n_warps; w0 += 8) {      // eight loads in flight, then their prefixes
          int t[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) t[k] = (w0 + k < n_warps) ? hist[(w0 + k) * 256 + d] : 0;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            if (w0 + k < n_warps) hist[(w0 + k) * 256 + d] = run;
            run += t[k];
          }
        }
        digit_tot[d] = run;
      }
      __syncthreads();
      dev::block_exclusive_scan(digit_tot, 256, warp_tot);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (dig[e] < 256) dst[digit_tot[dig[e]] + hist[warp * 256 + dig[e]] + loc[e]] = word[e];
      }
      __syncthreads();
      unsigned* t = src; src = dst; dst = t;
    }
    for (int r = tid; r < n_items; r += nthr) emit(r, int(src[r] & 0xffffu));
    finish();
    return;
  }

  if (n_items > kDevPlanRankLoopMax) {
    // ---- many items, some of 2^16 tokens or more: a bitonic sort of (length, index) pairs in shared memory, longest first, ties by index (which
    // is the (b, j) order).  n log^2 n compare-exchanges against the n^2 comparisons of the ranking loop below.
    int n2 = 1;
    while (n2 < n_items) n2 <<= 1;                       // <= cap: cap is four times the thread count
    int* key = it_len;
    int* idx = aux;                                      // the flags in aux were last read before the barrier above
    for (int i = tid; i < n2; i += nthr) {
      if (i >= n_items) key[i] = -1;                     // padding sorts after every item
      idx[i] = i;
    }
    __syncthreads();
    for (int k = 2; k <= n2; k <<= 1) {
      for (int j = k >> 1; j > 0; j >>= 1) {
        for (int t = tid; t < (n2 >> 1); t += nthr) {
          const int lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));
          const int hi = lo | j;
          const int kl = key[lo], kh = key[hi], il = idx[lo], ih = idx[hi];
          const bool hi_first = kh > kl || (kh == kl && ih < il);    // the element at `hi` belongs before the one at `lo`
          const bool forward = (lo & k) == 0;                        // this run is sorted first-to-last
          if (hi_first == forward) {
            key[lo] = kh; key[hi] = kl;
            idx[lo] = ih; idx[hi] = il;
          }
        }
        __syncthreads();
      }
    }
    for (int r = tid; r < n_items; r += nthr) emit(r, idx[r]);
    finish();
    return;
  }

  // ---- longest first, ties in (b, j) order: the rank of item i is the number of items before it
  const int4* len4 = reinterpret_cast<const int4*>(it_len);
  const int n_quads = (n_items + 3) >> 2;
  for (int i = tid; i < n_items; i += nthr) {
    const int len = it_len[i];
    int rank = 0;
#pragma unroll 4
    for (int k4 = 0; k4 < n_quads; ++k4) {   // four lengths per load, independent of each other: the loop is not a chain of loads
      const int4 x = len4[k4];
      const int k = 4 * k4;
      rank += (x.x > len || (x.x == len && k < i)) ? 1 : 0;
      rank += (x.y > len || (x.y == len && k + 1 < i)) ? 1 : 0;
      rank += (x.z > len || (x.z == len && k + 2 < i)) ? 1 : 0;
      rank += (x.w > len || (x.w == len && k + 3 < i)) ? 1 : 0;
    }
    emit(rank, i);
  }
  finish();
}

}  // namespace libra
