// The paper's two rollout-side schedulers as plain host code (no GPU): the heterogeneous-TP partition
// DP of the Global Resource Planner (Section 4.3, Algorithm 1 "RolloutDP") and the causality-aware
// prefix tree with its cost-benefit routing rule (Section 5).  C ABI in include/libra.h.
#include <algorithm>
#include <cstdint>
#include <limits>
#include <map>
#include <memory>
#include <vector>

#include "libra.h"

namespace {

// Cost(tp, first, last) of one inference instance serving a contiguous segment of the length-sorted
// requests.  The paper takes it from its Cost Evaluator, fitted by profiling (Section 4.6: linear
// operators O(L), attention T(L) = gamma L^2 + eta L + theta); here the same polynomial form is a
// parameter: a * sum(L) + b * sum(L^2) + c * count + d per degree, 0 for an empty segment.
struct SegmentCost {
  const double* coef;  // [n_tp][4]
  std::vector<double> s1, s2;  // prefix sums of L and L^2 over the sorted requests
  double operator()(int tp_index, int first, int last) const {  // 1-based, inclusive; first > last = empty
    if (first > last) return 0.0;
    const double* c = coef + 4 * tp_index;
    return c[0] * (s1[last] - s1[first - 1]) + c[1] * (s2[last] - s2[first - 1]) + c[2] * double(last - first + 1) + c[3];
  }
};

struct TrieNode {
  std::vector<int64_t> hist;           // residual-length counts per bin
  std::map<int32_t, int32_t> children;  // return-state label -> node index
};

}  // namespace

struct libra_trie_s {
  std::vector<int32_t> bin_upper;              // bin k holds lengths <= bin_upper[k] (last bin: everything above)
  std::vector<TrieNode> nodes;                 // node 0 unused; roots are per prompt
  std::map<int64_t, int32_t> roots;            // prompt id -> node index
  int bin_of(int64_t len) const {
    const int K = int(bin_upper.size()) + 1;
    for (int k = 0; k + 1 < K; ++k)
      if (len <= bin_upper[k]) return k;
    return K - 1;
  }
  int32_t new_node() {
    nodes.emplace_back();
    nodes.back().hist.assign(bin_upper.size() + 1, 0);
    return int32_t(nodes.size() - 1);
  }
};

namespace {

// dp[g][i] = best makespan of "exactly g GPUs serve the first i sorted requests" (Section 4.3):
//   dp[g][i] = min over tp <= g, 0 <= x <= i of max(dp[g - tp][i - x], Cost(tp, i - x + 1, i))
// Ties go to the earlier degree, then to the smaller x.
// When no cost coefficient is negative, the minimum over x is found without trying every x: as x grows the first
// term cannot grow (fewer requests left for the other instances) and the second cannot shrink (more requests on this
// one), so the minimum of their maximum sits where they cross; one bisection finds the crossing and a second one the
// leftmost x of the same value.  With a negative coefficient nothing is monotone and the states are relaxed forwards
// instead (every state offers max(its value, cost of the next segment) to its successors; the smallest
// (value, degree, x) wins).
int rollout_dp_impl(int32_t n_gpus, const int32_t* lengths, int32_t n_requests, const int32_t* tp_set,
                    int32_t n_tp, const double* cost_coef, double* makespan, int32_t* inst_tp, int32_t* inst_first,
                    int32_t* inst_count, int32_t inst_capacity, int32_t* n_instances) {
  if (n_gpus < 0 || n_requests < 0 || n_tp <= 0 || !tp_set || !cost_coef || !makespan || !n_instances) {
    return LIBRA_INVALID_ARGUMENT;
  }
  if (n_requests > 0 && !lengths) return LIBRA_INVALID_ARGUMENT;
  for (int t = 0; t < n_tp; ++t)
    if (tp_set[t] <= 0) return LIBRA_INVALID_ARGUMENT;
  const int G = n_gpus, L = n_requests;
  std::vector<int32_t> sorted(lengths, lengths + L);
  std::sort(sorted.begin(), sorted.end());  // non-decreasing: every instance gets a contiguous segment
  bool monotone = true;
  for (int t = 0; t < 4 * n_tp; ++t) monotone = monotone && cost_coef[t] >= 0.0;
  for (int i = 0; i < L; ++i) monotone = monotone && sorted[size_t(i)] >= 0;
  SegmentCost cost;
  cost.coef = cost_coef;
  cost.s1.assign(L + 1, 0.0);
  cost.s2.assign(L + 1, 0.0);
  for (int i = 1; i <= L; ++i) {
    cost.s1[i] = cost.s1[i - 1] + double(sorted[i - 1]);
    cost.s2[i] = cost.s2[i - 1] + double(sorted[i - 1]) * double(sorted[i - 1]);
  }
  const double inf = std::numeric_limits<double>::infinity();
  const size_t W = size_t(L) + 1;
  std::vector<double> dp((size_t(G) + 1) * W, inf);
  std::vector<int32_t> arg_tp((size_t(G) + 1) * W, -1), arg_x((size_t(G) + 1) * W, -1);
  dp[0] = 0.0;  // dp[0][0]
  if (!monotone) {
    // forward relaxation; dp[g'][.] is final once every g < g' has been expanded, because degrees are positive
    for (int g = 0; g < G; ++g) {
      for (int i = 0; i <= L; ++i) {
        const double here = dp[size_t(g) * W + i];
        if (here == inf) continue;
        for (int t = 0; t < n_tp; ++t) {
          const int g2 = g + tp_set[t];
          if (g2 > G) continue;
          for (int x = 0; i + x <= L; ++x) {
            const double v = std::max(here, cost(t, i + 1, i + x));
            const size_t at = size_t(g2) * W + size_t(i + x);
            const bool better = v < dp[at] || (v == dp[at] && (t < arg_tp[at] || (t == arg_tp[at] && x < arg_x[at])));
            if (better) {
              dp[at] = v;
              arg_tp[at] = t;
              arg_x[at] = x;
            }
          }
        }
      }
    }
  }
  for (int g = 1; monotone && g <= G; ++g) {
    for (int i = 0; i <= L; ++i) {
      double best = inf;
      int btp = -1, bx = -1;
      for (int t = 0; t < n_tp; ++t) {
        const int tp = tp_set[t];
        if (tp > g) continue;
        const double* prev = &dp[size_t(g - tp) * W];
        // first x at which this instance's cost reaches what the others need (x = i + 1 if it never does)
        int lo = 0, hi = i + 1;
        while (lo < hi) {
          const int mid = (lo + hi) / 2;
          if (cost(t, i - mid + 1, i) >= prev[i - mid]) hi = mid;
          else lo = mid + 1;
        }
        double cand = inf;
        int cx = -1;
        for (int x = std::max(0, lo - 1); x <= std::min(i, lo); ++x) {   // the two sides of the crossing
          const double v = std::max(prev[i - x], cost(t, i - x + 1, i));
          if (v < cand) {
            cand = v;
            cx = x;
          }
        }
        if (cx < 0 || !(cand < best)) continue;
        // the leftmost x with the same value: left of the crossing the maximum is prev[i - x], which does not grow
        int l2 = 0, h2 = cx;
        while (l2 < h2) {
          const int mid = (l2 + h2) / 2;
          if (prev[i - mid] <= cand) h2 = mid;
          else l2 = mid + 1;
        }
        best = cand;
        btp = t;
        bx = l2;
      }
      dp[size_t(g) * W + i] = best;
      arg_tp[size_t(g) * W + i] = btp;
      arg_x[size_t(g) * W + i] = bx;
    }
  }
  *makespan = dp[size_t(G) * W + L];
  *n_instances = 0;
  if (*makespan == inf) return LIBRA_OK;  // no partition uses exactly n_gpus GPUs (reported as +inf)
  // backtrack: instances from the last (longest requests) to the first
  int g = G, i = L, count = 0;
  std::vector<int32_t> tps, firsts, counts;
  while (g > 0) {
    const int t = arg_tp[size_t(g) * W + i], x = arg_x[size_t(g) * W + i];
    tps.push_back(tp_set[t]);
    firsts.push_back(i - x);  // 0-based index of the segment's first request in the sorted list
    counts.push_back(x);
    g -= tp_set[t];
    i -= x;
    ++count;
  }
  *n_instances = count;
  if (count > inst_capacity) return LIBRA_WORKSPACE_TOO_SMALL;
  if (count > 0 && (!inst_tp || !inst_first || !inst_count)) return LIBRA_INVALID_ARGUMENT;
  for (int k = 0; k < count; ++k) {  // in sorted-request order
    inst_tp[k] = tps[size_t(count - 1 - k)];
    inst_first[k] = firsts[size_t(count - 1 - k)];
    inst_count[k] = counts[size_t(count - 1 - k)];
  }
  return LIBRA_OK;
}

}  // namespace

extern "C" {

int libra_rollout_dp(int32_t n_gpus, const int32_t* lengths, int32_t n_requests, const int32_t* tp_set, int32_t n_tp,
                     const double* cost_coef, double* makespan, int32_t* inst_tp, int32_t* inst_first,
                     int32_t* inst_count, int32_t inst_capacity, int32_t* n_instances) {
  return rollout_dp_impl(n_gpus, lengths, n_requests, tp_set, n_tp, cost_coef, makespan, inst_tp, inst_first, inst_count,
                         inst_capacity, n_instances);
}

int libra_trie_create(libra_trie_t* trie, const int32_t* bin_upper, int32_t n_thresholds) {
  if (!trie) return LIBRA_INVALID_ARGUMENT;
  *trie = nullptr;
  if (n_thresholds < 0 || (n_thresholds > 0 && !bin_upper)) return LIBRA_INVALID_ARGUMENT;
  for (int k = 1; k < n_thresholds; ++k)
    if (bin_upper[k] <= bin_upper[k - 1]) return LIBRA_INVALID_ARGUMENT;
  libra_trie_s* t = new (std::nothrow) libra_trie_s();
  if (!t) return LIBRA_INVALID_ARGUMENT;
  t->bin_upper.assign(bin_upper, bin_upper + n_thresholds);
  t->nodes.emplace_back();  // index 0: sentinel
  *trie = t;
  return LIBRA_OK;
}

int libra_trie_destroy(libra_trie_t trie) {
  delete trie;
  return LIBRA_OK;
}

int libra_trie_insert(libra_trie_t t, int64_t prompt_id, const int32_t* states, int32_t n_states,
                      const int32_t* residual_lengths) {
  if (!t || n_states < 0 || !residual_lengths || (n_states > 0 && !states)) return LIBRA_INVALID_ARGUMENT;
  for (int k = 0; k <= n_states; ++k)
    if (residual_lengths[k] < 0) return LIBRA_INVALID_ARGUMENT;
  auto it = t->roots.find(prompt_id);
  int32_t node = (it == t->roots.end()) ? (t->roots[prompt_id] = t->new_node()) : it->second;
  t->nodes[size_t(node)].hist[size_t(t->bin_of(residual_lengths[0]))] += 1;  // at the root: the whole remaining length
  for (int k = 0; k < n_states; ++k) {
    auto& ch = t->nodes[size_t(node)].children;
    auto c = ch.find(states[k]);
    int32_t next;
    if (c == ch.end()) {
      next = t->new_node();
      t->nodes[size_t(node)].children[states[k]] = next;  // (re-index: new_node may have moved the vector)
    } else {
      next = c->second;
    }
    node = next;
    t->nodes[size_t(node)].hist[size_t(t->bin_of(residual_lengths[k + 1]))] += 1;
  }
  return LIBRA_OK;
}

int libra_trie_lookup(libra_trie_t t, int64_t prompt_id, const int32_t* states, int32_t n_states, double* hist,
                      int32_t* depth_reached, int64_t* samples) {
  if (!t || n_states < 0 || !hist || (n_states > 0 && !states)) return LIBRA_INVALID_ARGUMENT;
  const int K = int(t->bin_upper.size()) + 1;
  for (int k = 0; k < K; ++k) hist[k] = 0.0;
  if (depth_reached) *depth_reached = -1;
  if (samples) *samples = 0;
  auto it = t->roots.find(prompt_id);
  if (it == t->roots.end()) return LIBRA_OK;  // unknown prompt: empty distribution, depth -1
  int32_t node = it->second;
  int depth = 0;
  for (int k = 0; k < n_states; ++k) {  // an unseen state: stay at the parent (back-off)
    const auto& ch = t->nodes[size_t(node)].children;
    auto c = ch.find(states[k]);
    if (c == ch.end()) break;
    node = c->second;
    ++depth;
  }
  int64_t total = 0;
  for (int k = 0; k < K; ++k) total += t->nodes[size_t(node)].hist[size_t(k)];
  for (int k = 0; k < K; ++k) hist[k] = total ? double(t->nodes[size_t(node)].hist[size_t(k)]) / double(total) : 0.0;
  if (depth_reached) *depth_reached = depth;
  if (samples) *samples = total;
  return LIBRA_OK;
}

int libra_trie_route(libra_trie_t t, int64_t prompt_id, const int32_t* states, int32_t n_states, int32_t n_buckets,
                     const double* decode_cost, const double* migration_cost, int32_t* best_bucket, double* best_cost) {
  if (!t || n_buckets <= 0 || !decode_cost || !migration_cost || !best_bucket) return LIBRA_INVALID_ARGUMENT;
  const int K = int(t->bin_upper.size()) + 1;
  std::vector<double> p(size_t(K), 0.0);
  int32_t depth = -1;
  int64_t samples = 0;
  const int rc = libra_trie_lookup(t, prompt_id, states, n_states, p.data(), &depth, &samples);
  if (rc != LIBRA_OK) return rc;
  // B* = argmin_B ( sum_k p_k * Tdec(B, k) + Cmig(B_cur, B) ); ties go to the lower bucket index
  double best = std::numeric_limits<double>::infinity();
  int arg = -1;
  for (int b = 0; b < n_buckets; ++b) {
    double c = migration_cost[b];
    for (int k = 0; k < K; ++k) c += p[size_t(k)] * decode_cost[size_t(b) * K + k];
    if (c < best) {
      best = c;
      arg = b;
    }
  }
  *best_bucket = arg;
  if (best_cost) *best_cost = best;
  return LIBRA_OK;
}

}  // extern "C"
