#include "planner.hpp"

#include "plan_layout.hpp"

#include <algorithm>

namespace libra {
namespace {
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }
inline int64_t next_pow2(int64_t x) {
  int64_t r = 1;
  while (r < x) r <<= 1;
  return r;
}
inline int32_t log2_exact(int64_t x) {
  int32_t k = 0;
  while ((int64_t(1) << k) < x) ++k;
  return k;
}
}  // namespace

bool valid_params(const PlanParams& p) {
  if (p.n_sm <= 0 || p.ctas_per_sm <= 0 || p.items_per_slot <= 0) return false;
  if (p.chunk_align <= 0 || p.chunk_align % 16 != 0) return false;
  if (p.min_chunk <= 0) return false;
  if (p.max_splits <= 0 || p.max_splits > 64 || (p.max_splits & (p.max_splits - 1)) != 0) return false;
  if (p.refine != 0 && p.refine != 1) return false;
  return true;
}

int64_t max_items(const PlanParams& p, int32_t num_kv_heads, int32_t max_batch) {
  const int64_t slots = int64_t(p.n_sm) * p.ctas_per_sm * p.items_per_slot;
  const int64_t plain = 2 * ceil_div(slots, num_kv_heads) + max_batch;
  if (!p.refine) return plain;
  // a plan is made again for 2 * slots only when it had fewer than 1.5 waves of blocks, i.e. fewer than
  // 1.5 * W / Hkv items, hence non-empty sequences
  const int64_t wave = int64_t(p.n_sm) * p.ctas_per_sm;
  const int64_t few = std::min<int64_t>(max_batch, (plan_layout::kRefineWavesNum * wave) / (plan_layout::kRefineWavesDen * num_kv_heads));
  return std::max(plain, 2 * ceil_div(2 * slots, num_kv_heads) + few);
}

bool make_plan(const PlanParams& p, int32_t num_kv_heads, const int32_t* seq_lens, int32_t batch, HostPlan* out) {
  if (!valid_params(p) || num_kv_heads <= 0 || batch < 0 || out == nullptr) return false;
  int64_t total = 0;
  for (int32_t b = 0; b < batch; ++b) {
    if (seq_lens[b] < 0) return false;
    total += seq_lens[b];
  }
  const int64_t slots = int64_t(p.n_sm) * p.ctas_per_sm * p.items_per_slot;
  int64_t base = std::max<int64_t>(p.min_chunk, round_up(ceil_div(int64_t(num_kv_heads) * total, slots), p.chunk_align));

  HostPlan& pl = *out;
  pl.batch = batch;
  pl.bucket.assign(batch, -1);
  pl.num_splits.assign(batch, 0);
  pl.chunk_len.assign(batch, 0);
  pl.item_offset.assign(batch, 0);
  pl.items.clear();
  pl.combine.clear();
  pl.empty.clear();

  // buckets for a base length; returns the number of work items
  auto bucket_all = [&](int64_t base_len) -> int64_t {
    int64_t n_items = 0;
    for (int32_t b = 0; b < batch; ++b) {
      const int64_t len = seq_lens[b];
      if (len == 0) continue;
      int64_t degree = next_pow2(ceil_div(len, base_len));
      if (base_len < plan_layout::kSmallBaseTokens && degree > 1 &&
          len * plan_layout::kGeoMeanDen < (degree / 2) * base_len * plan_layout::kGeoMeanNum) {
        degree /= 2;   // short chunks: the nearer power of two, see plan_layout.hpp
      }
      degree = std::min<int64_t>(degree, p.max_splits);
      const int64_t chunk = round_up(ceil_div(len, degree), p.chunk_align);
      const int64_t pieces = ceil_div(len, chunk);
      pl.bucket[b] = log2_exact(degree);
      pl.chunk_len[b] = int32_t(chunk);
      pl.num_splits[b] = int32_t(pieces);
      n_items += pieces;
    }
    return n_items;
  };
  const int64_t n_items = bucket_all(base);
  // A coarse plan of long blocks - fewer than one and a half waves of the resident blocks - is made again for twice
  // as many slots: with so few blocks most SMs idle through the second wave and the rest cannot pull the memory
  // bandwidth alone (plan_layout.hpp).
  const int64_t wave = int64_t(p.n_sm) * p.ctas_per_sm;
  if (p.refine && base >= plan_layout::kRefineMinBaseTokens &&
      plan_layout::kRefineWavesDen * num_kv_heads * n_items < plan_layout::kRefineWavesNum * wave) {
    base = std::max<int64_t>(p.min_chunk, round_up(ceil_div(int64_t(num_kv_heads) * total, 2 * slots), p.chunk_align));
    bucket_all(base);
  }
  pl.chunk_target = int32_t(base);

  int32_t running = 0;
  for (int32_t b = 0; b < batch; ++b) {
    const int64_t len = seq_lens[b];
    pl.item_offset[b] = running;
    if (len == 0) {
      pl.empty.push_back(b);
      continue;
    }
    const int64_t chunk = pl.chunk_len[b];
    const int64_t pieces = pl.num_splits[b];
    for (int64_t j = 0; j < pieces; ++j) {
      pl.items.push_back(WorkItem{b, int32_t(j), int32_t(j * chunk), int32_t(std::min(len, (j + 1) * chunk))});
    }
    if (pieces > 1) pl.combine.push_back(b);
    running += int32_t(pieces);
  }
  // longest first; items were generated in (b, j) order, so a stable sort keeps that order among equals
  std::stable_sort(pl.items.begin(), pl.items.end(), [](const WorkItem& x, const WorkItem& y) {
    return (x.kv_end - x.kv_begin) > (y.kv_end - y.kv_begin);
  });
  return true;
}

}  // namespace libra
