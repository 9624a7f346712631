// Layout of the plan as uploaded into the device workspace (all int32), shared by the host code
// that writes it and the kernels that read it.
//
//   [0, 16)                      header (see indices below); word kErrorWord is the device error word
//   [16, 16 + 4*num_items)       work items, longest first: {b | j << 18 | n_b << 24, kv_begin, kv_end, slot}
//                                slot = item_offset[b] + j if the sequence is split, else -1
//   [combine_off, +4*num_fix)    fix-up entries: {b, first_slot, n, planned_len}; n > 1: merge n
//                                partial results; n == 0: empty sequence, write zeros
#pragma once
#include <cstdint>

namespace libra {
namespace plan_layout {
constexpr int kHeaderInts = 16;
constexpr int kItemInts = 4;
constexpr int kFixInts = 4;
constexpr int kMagicValue = 0x4c425241;  // "LBRA"
// header word indices
constexpr int kMagic = 0;
constexpr int kBatch = 1;
constexpr int kNumItems = 2;
constexpr int kNumFix = 3;
constexpr int kFixOff = 4;     // int offset of the fix-up entries from the start of the blob
constexpr int kNumCombine = 5; // the first kNumCombine fix-up entries are merges, the rest empty sequences
constexpr int kErrorWord = 8;
// packing of word 0 of a work item: sequence index, chunk index j, chunk count n_b (<= 64)
constexpr int kChunkShift = 18;
constexpr int kCountShift = 24;
constexpr int kMaxBatch = 1 << kChunkShift;
}  // namespace plan_layout
}  // namespace libra

#define LIBRA_DEV_ERR_WAIT_TIMEOUT 1u
#define LIBRA_DEV_ERR_BAD_PAGE_ID 2u
#define LIBRA_DEV_ERR_SEQ_LEN_MISMATCH 4u
