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
  if (p.wave_fill < 0 || p.wave_fill > 2) return false;   // max_items() covers two waves
  return true;
}

int64_t max_items(const PlanParams& p, int32_t num_kv_heads, int32_t max_batch) {
  const int64_t slots = int64_t(p.n_sm) * p.ctas_per_sm * p.items_per_slot;
  return 2 * ceil_div(slots, num_kv_heads) + max_batch;
}

bool make_plan(const PlanParams& p, int32_t num_kv_heads, const int32_t* seq_lens, int32_t batch, HostPlan* out) {
  if (!valid_params(p) || num_kv_heads <= 0 || batch < 0 || out == nullptr) return false;
  int64_t total = 0;
  for (int32_t b = 0; b < batch; ++b) {
    if (seq_lens[b] < 0) return false;
    total += seq_lens[b];
  }
  const int64_t slots = int64_t(p.n_sm) * p.ctas_per_sm * p.items_per_slot;
  const int64_t base = std::max<int64_t>(p.min_chunk, round_up(ceil_div(int64_t(num_kv_heads) * total, slots), p.chunk_align));

  HostPlan& pl = *out;
  pl.batch = batch;
  pl.chunk_target = int32_t(base);
  pl.bucket.assign(batch, -1);
  pl.num_splits.assign(batch, 0);
  pl.chunk_len.assign(batch, 0);
  pl.item_offset.assign(batch, 0);
  pl.items.clear();
  pl.combine.clear();
  pl.empty.clear();

  for (int32_t b = 0; b < batch; ++b) {
    const int64_t len = seq_lens[b];
    if (len == 0) continue;
    int64_t degree = next_pow2(ceil_div(len, base));
    if (base < plan_layout::kSmallBaseTokens && degree > 1 &&
        len * plan_layout::kGeoMeanDen < (degree / 2) * base * plan_layout::kGeoMeanNum) {
      degree /= 2;   // short chunks: the nearer power of two, see plan_layout.hpp
    }
    degree = std::min<int64_t>(degree, p.max_splits);
    const int64_t chunk = round_up(ceil_div(len, degree), p.chunk_align);
    const int64_t pieces = ceil_div(len, chunk);
    pl.bucket[b] = log2_exact(degree);
    pl.chunk_len[b] = int32_t(chunk);
    pl.num_splits[b] = int32_t(pieces);
  }

  // Wave fill.  The launch is `blocks` thread blocks on `wave` resident ones.  When that is at most wave_fill waves,
  // the slots the last wave leaves free are handed out as extra chunks, one each to the sequences with the longest
  // chunks (ties: lower index first): a few equally long sequences otherwise run one full wave and one part-empty
  // wave of equally long blocks.  The bucket of a sequence (its length class) stays.
  const int64_t wave = int64_t(p.n_sm) * p.ctas_per_sm;
  int64_t blocks = 0;
  for (int32_t b = 0; b < batch; ++b) blocks += int64_t(num_kv_heads) * pl.num_splits[b];
  const int64_t waves = ceil_div(blocks, wave);
  if (waves >= 1 && waves <= p.wave_fill) {
    const int64_t spare = (waves * wave - blocks) / num_kv_heads;
    std::vector<int32_t> order;
    for (int32_t b = 0; b < batch; ++b)
      if (seq_lens[b] > 0) order.push_back(b);
    const size_t take = size_t(std::min<int64_t>(spare, int64_t(order.size())));
    std::partial_sort(order.begin(), order.begin() + take, order.end(), [&](int32_t x, int32_t y) {
      return pl.chunk_len[x] != pl.chunk_len[y] ? pl.chunk_len[x] > pl.chunk_len[y] : x < y;
    });
    for (size_t i = 0; i < take; ++i) {
      const int32_t b = order[i];
      const int64_t len = seq_lens[b];
      const int64_t chunk = round_up(ceil_div(len, int64_t(pl.num_splits[b]) + 1), p.chunk_align);
      if (chunk < p.min_chunk || pl.num_splits[b] + 1 > p.max_splits) continue;
      pl.chunk_len[b] = int32_t(chunk);
      pl.num_splits[b] = int32_t(ceil_div(len, chunk));
    }
  }

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
