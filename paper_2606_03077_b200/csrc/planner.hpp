// Length-bucketed work planner (host, integers only).
//
// Mirrors, inside one GPU, the bucket idea of the paper's rollout scheduler (Section 2.3: one
// parallel degree per length range; Section 4.3: degrees are powers of two, requests sorted by
// length, minimise the maximum completion time; Section 5: buckets ordered by capacity, bins
// aligned with the bucket thresholds).  A sequence's "degree" here is the number of thread blocks
// that share its KV range.
#pragma once
#include <cstdint>
#include <vector>

namespace libra {

struct PlanParams {
  int32_t n_sm = 148;
  int32_t ctas_per_sm = 1;
  int32_t items_per_slot = 1;
  int32_t chunk_align = 256;
  int32_t min_chunk = 512;
  int32_t max_splits = 64;
  int32_t refine = 1;      // 1: a plan of fewer than 1.5 waves of long blocks is made again twice as fine (0 = never)
};

struct WorkItem {  // one (sequence, chunk) unit; the decode grid is items x KV heads
  int32_t b, j, kv_begin, kv_end;
};

struct HostPlan {
  int32_t batch = 0;
  int32_t chunk_target = 0;
  std::vector<int32_t> bucket, num_splits, chunk_len, item_offset;
  std::vector<WorkItem> items;  // longest first
  std::vector<int32_t> combine, empty;
};

// false if params are unusable or a length is negative
bool valid_params(const PlanParams& p);
bool make_plan(const PlanParams& p, int32_t num_kv_heads, const int32_t* seq_lens, int32_t batch, HostPlan* out);

// Upper bound of the number of work items for any batch <= max_batch:
// n_b <= 2*cd(L_b, C) - 1 and C >= num_kv_heads*T/(W*items_per_slot) give sum n_b <= 2*cd(W*ips, Hkv) + B;
// a refined plan is a plan for 2*W*ips slots of a batch with fewer than 1.5*W/Hkv non-empty sequences (else it would
// not have been refined): sum n_b <= 2*cd(2*W*ips, Hkv) + min(B, 1.5*W/Hkv).  The bound is the larger of the two.
int64_t max_items(const PlanParams& p, int32_t num_kv_heads, int32_t max_batch);

}  // namespace libra
