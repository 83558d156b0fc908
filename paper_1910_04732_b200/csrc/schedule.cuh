// Static tile schedule of a grouped GEMM launch.
//
// A grouped launch walks one work list (the tiles of all its problems) with a fixed set of
// persistent units (CTAs, or CTA pairs).  Dealing the list out round-robin gives every unit the
// same NUMBER of tiles, which is only balanced when the tiles cost the same.  The launches of the
// gated factorized layer mix tiles of different length: in H' = X Q^T and dH' = dY P the FFN
// matrices contract over 3072 features (48 k-blocks) next to attention matrices that contract
// over 768 (12 k-blocks).  The host therefore assigns tiles to units with the longest-processing-time rule (sort by cost,
// always hand the next tile to the least loaded unit) and passes the per-unit lists to the kernel
// as a table in its parameter block; every role of a unit (TMA producer, MMA issuer, epilogue
// warps, and both CTAs of a pair) walks the same list, so no run-time hand-over is needed.
// Launches with more work items than the table holds keep the round-robin order (with that many
// tiles per unit the imbalance is small anyway).
#pragma once
#include <stdint.h>

#ifndef __CUDACC_RTC__
#include <algorithm>
#include <functional>
#include <queue>
#include <utility>
#include <vector>
#endif

namespace flop {
namespace tc {

constexpr int kMaxSched = 2048;   // work items a table can hold
constexpr int kSchedProblemShift = 11;   // grouped launches: entry = (problem index << 11) | work-list index
constexpr int kMaxUnits = 148;    // persistent CTAs (one-CTA kernel) or pairs (two-CTA kernel)

struct Schedule {
  int n_units;                       // 0: no table, round-robin over the work list
  uint16_t begin[kMaxUnits + 1];     // unit u walks item[begin[u] .. begin[u+1])
  uint16_t item[kMaxSched];          // work-list indices
};

// Longest-processing-time assignment of `cost.size()` work items to `units` units.  Items of equal
// cost keep their work-list order (neighbouring tiles share operand tiles in L2).  Returns the
// largest unit load; `rr_makespan` receives the largest load of the round-robin deal for comparison.
inline double build_schedule(const std::vector<double>& cost, int units, Schedule* out, double* rr_makespan) {
  const int n = (int)cost.size();
  out->n_units = 0;
  if (rr_makespan) {
    std::vector<double> load((size_t)std::max(units, 1), 0.0);
    for (int i = 0; i < n; ++i) load[(size_t)(i % std::max(units, 1))] += cost[(size_t)i];
    *rr_makespan = load.empty() ? 0.0 : *std::max_element(load.begin(), load.end());
  }
  if (n == 0 || n > kMaxSched || units <= 0 || units > kMaxUnits) return -1.0;
  if (rr_makespan) {
    // Nothing to gain when round-robin is already within 3 % of the lower bound max(mean load, longest item):
    // skip the sort (this keeps the host cost of the common equal-tile launches at one pass over the list).
    double total = 0.0, longest = 0.0;
    for (int i = 0; i < n; ++i) { total += cost[(size_t)i]; longest = std::max(longest, cost[(size_t)i]); }
    if (*rr_makespan <= 1.03 * std::max(total / units, longest)) return -1.0;
  }
  std::vector<int> order((size_t)n);
  for (int i = 0; i < n; ++i) order[(size_t)i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cost[(size_t)a] > cost[(size_t)b]; });
  typedef std::pair<double, int> LoadUnit;   // least loaded first, ties to the lower unit index
  std::priority_queue<LoadUnit, std::vector<LoadUnit>, std::greater<LoadUnit>> heap;
  for (int u = 0; u < units; ++u) heap.push(LoadUnit(0.0, u));
  std::vector<std::vector<int>> lists((size_t)units);
  double makespan = 0.0;
  for (int i = 0; i < n; ++i) {
    LoadUnit lu = heap.top();
    heap.pop();
    lists[(size_t)lu.second].push_back(order[(size_t)i]);
    lu.first += cost[(size_t)order[(size_t)i]];
    makespan = std::max(makespan, lu.first);
    heap.push(lu);
  }
  int pos = 0;
  for (int u = 0; u < units; ++u) {
    out->begin[u] = (uint16_t)pos;
    for (int w : lists[(size_t)u]) out->item[pos++] = (uint16_t)w;
  }
  for (int u = units; u <= kMaxUnits; ++u) out->begin[u] = (uint16_t)pos;
  out->n_units = units;
  return makespan;
}

// Queue of a chained launch (gemm_tc2_chain.cuh): the work list holds the tiles of two stages, a tile of the
// second stage waits for first-stage tiles, and the persistent units draw tiles from the head of one queue.
// All first-stage tiles must therefore come before all second-stage tiles (a drawn tile then only waits for
// tiles that some unit already works on, so no wait can be circular).  Inside a stage the queue follows `key`
// (ties keep list order): the caller puts first what other tiles wait for, long tiles before short ones, and
// orders consumers like their producers.  out->item holds the queue (n_units = 1 marks the table as valid).
// Returns false when the table cannot hold the launch (the kernel then walks the work list in its own order,
// which the caller keeps stage-ordered).
inline bool build_chain_queue(const std::vector<int>& stage, const std::vector<int64_t>& key, Schedule* out) {
  const int n = (int)stage.size();
  out->n_units = 0;
  if (n == 0 || n > kMaxSched || (int)key.size() != n) return false;
  std::vector<int> order((size_t)n);
  for (int i = 0; i < n; ++i) order[(size_t)i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
    const int sa = stage[(size_t)a] != 0, sb = stage[(size_t)b] != 0;
    if (sa != sb) return sa < sb;
    return key[(size_t)a] < key[(size_t)b];
  });
  for (int i = 0; i < n; ++i) out->item[i] = (uint16_t)order[(size_t)i];
  out->begin[0] = 0;
  for (int u = 1; u <= kMaxUnits; ++u) out->begin[u] = (uint16_t)n;
  out->n_units = 1;
  return true;
}

}  // namespace tc
}  // namespace flop
