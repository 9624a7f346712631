// The plan as the kernels see it (shared by the host code that writes it and the kernels that read it).
//
//   entries[0 .. num_items)              work items, longest first:
//                                        {b | j << 18 | n_b << 24, kv_begin, kv_end, slot}
//                                        slot = item_offset[b] + j if the sequence is split, else -1
//   entries[num_items .. +num_empty)     one entry {b, 0, 0, 0} per empty sequence
//   fixes[0 .. num_combine)              merges for the combine kernel: {b, first_slot, n_b, planned_len}
//
// Plans of up to kParamEntries entries (and kParamFixEntries merges) do not go through device memory
// at all: they are passed to the kernels by value as a kernel parameter, which saves the upload and
// its place in the stream.  Larger plans are uploaded into the workspace in the same format, and the
// device-side planner writes its plan there too, preceded by kCountInts counts that the kernels read.
#pragma once
#include <cstdint>

#include <vector_types.h>

namespace libra {
namespace plan_layout {
// packing of word 0 of a work item: sequence index, chunk index j, chunk count n_b (<= 64)
constexpr int kChunkShift = 18;
constexpr int kCountShift = 24;
constexpr int kMaxBatch = 1 << kChunkShift;
constexpr int kParamEntries = 768;  // 12 KB of the 32 KB kernel-parameter space
constexpr int kParamFixEntries = 256;
// Split degree of a sequence (both planners): the least power of two >= ceil(len / base) - except that, when the base
// chunk is shorter than kSmallBaseTokens, the power of two below it is taken if len / base is nearer to it in ratio
// (below the geometric mean of the two: len * 128 < (degree / 2) * base * 181, 181 / 128 ~ sqrt 2).  A unit costs
// ~4 us of start-up and epilogue whatever its length; on chunks that short, fewer and longer units win (measured
// 8 - 18 % on batches cut by KV head over 4 - 8 ranks, nothing lost elsewhere; with longer chunks the finer cut is
// the better one).
constexpr int kSmallBaseTokens = 4096;
constexpr int kGeoMeanNum = 181, kGeoMeanDen = 128;
// A plan with fewer than kRefineWavesNum / kRefineWavesDen waves of blocks whose base chunk is at least
// kRefineMinBaseTokens long is made again for twice as many slots (both planners).  Few long blocks leave most SMs idle
// through the last wave, and the blocks that do run cannot pull the memory bandwidth alone: 12 sequences of 20,000
// tokens 169 -> 147 us, 26 sequences of 16K - 32K tokens 420 -> 389 us, 3 of 40,000 89 -> 79 us; batches of 1.5 waves
// and more lose 1 - 3 % when cut finer, and on short bases the fixed cost of a block dominates.
constexpr int kRefineWavesNum = 3, kRefineWavesDen = 2;
constexpr int kRefineMinBaseTokens = 4096;
// counts written by the device-side planner (int32 words at the start of the workspace's plan region)
constexpr int kCountInts = 8;
constexpr int kCntItems = 0;
constexpr int kCntCombine = 1;
constexpr int kCntEmpty = 2;
constexpr int kCntChunkTarget = 3;
constexpr int kCntOverflow = 4;
}  // namespace plan_layout

struct ParamPlan {
  int4 e[plan_layout::kParamEntries];
};
struct ParamFix {  // merges for the stand-alone combine kernel: {b, first_slot, n, planned_len}
  int4 e[plan_layout::kParamFixEntries];
};
}  // namespace libra

#define LIBRA_DEV_ERR_WAIT_TIMEOUT 1u
#define LIBRA_DEV_ERR_BAD_PAGE_ID 2u
#define LIBRA_DEV_ERR_SEQ_LEN_MISMATCH 4u
#define LIBRA_DEV_ERR_PLAN_OVERFLOW 8u
