// Bit-width selection (Section 3.4, Eq. 5): for every layer one of two precisions, minimal summed perturbation
// Omega subject to limits on the summed model size, BOPS and latency.  Host code only: an exact depth-first
// branch and bound over the layers.
//
//   bound      For each active limit on its own the remaining layers form a fractional knapsack: start every
//              layer at its cheaper precision for that resource, then buy the upgrades (less Omega for more of the
//              resource) in order of Omega saved per unit until the budget is spent, the last one in part.  The
//              optimum of that relaxation is a lower bound on what the remaining layers can add to the objective
//              under all limits together; the largest of the (at most three) bounds is used.
//   pruning    a node is dropped when its bound cannot beat the best assignment found so far, or when even the
//              cheapest completion overshoots a limit.
//   order      layers with the largest Omega difference are decided first, the smaller Omega tried first.
//
// All quantities are integers (the caller picks the units: bytes, bit operations, nanoseconds, any fixed-point
// unit for Omega), so sums do not depend on their order and the result can be compared exactly with a plain
// enumeration of all assignments.
#include <algorithm>
#include <cstdint>
#include <vector>

#include "../../include/hq.h"

namespace {

constexpr int kRes = 3;                      // size, BOPS, latency
constexpr int64_t kMaxValue = 1LL << 40;     // per entry; with at most 4096 layers every sum stays below 2^52
constexpr long long kNodeBudget = 200000000; // the search gives up (HQ_ERR_UNSUPPORTED) beyond this many nodes

struct Problem {
  int n = 0;
  std::vector<int> order;                    // search position -> layer
  std::vector<int> pos_of;                   // layer -> search position
  std::vector<int64_t> om[2], rs[kRes][2];   // per layer, per choice
  int64_t limit[kRes];
  bool active[kRes];
  // per resource: the cheaper ("lo") and dearer ("hi") choice of every layer, the layers sorted by Omega saved per
  // unit of the resource (free upgrades first, upgrades that save nothing last), and suffix sums over the search order
  std::vector<int> lo[kRes], eff[kRes];
  std::vector<int64_t> suf_lo_om[kRes], suf_lo_rs[kRes];
  std::vector<int64_t> suf_min_om;           // no active limit: every layer takes its smaller Omega
  // search state
  std::vector<int> cur, best;
  int64_t best_obj = -1;                     // -1: nothing found yet
  long long nodes = 0;
  bool gave_up = false;
};

// Lower bound on the Omega the layers at search positions >= pos can add, given the resources already used.
// Returns -1 when no completion can meet the limits.
int64_t remaining_bound(const Problem& p, int pos, const int64_t (&used)[kRes]) {
  int64_t bound = -2;
  for (int r = 0; r < kRes; ++r) {
    if (!p.active[r]) continue;
    int64_t budget = p.limit[r] - used[r] - p.suf_lo_rs[r][pos];
    if (budget < 0) return -1;
    int64_t gain = 0;
    for (int layer : p.eff[r]) {
      if (p.pos_of[layer] < pos) continue;
      const int l = p.lo[r][layer], h = 1 - l;
      const int64_t d_om = p.om[l][layer] - p.om[h][layer];
      if (d_om <= 0) break;                                      // the rest saves nothing
      const int64_t d_rs = p.rs[r][h][layer] - p.rs[r][l][layer];
      if (d_rs <= budget) { gain += d_om; budget -= d_rs; continue; }
      gain += (int64_t)(((__int128)d_om * budget + d_rs - 1) / d_rs);   // the part that still fits, rounded up
      break;
    }
    const int64_t b = p.suf_lo_om[r][pos] - gain;
    if (b > bound) bound = b;
  }
  return bound == -2 ? p.suf_min_om[pos] : bound;
}

void search(Problem& p, int pos, int64_t (&used)[kRes], int64_t obj) {
  if (p.gave_up) return;
  if (++p.nodes > kNodeBudget) { p.gave_up = true; return; }
  if (pos == p.n) {
    if (p.best_obj < 0 || obj < p.best_obj) { p.best_obj = obj; p.best = p.cur; }
    return;
  }
  const int64_t rest = remaining_bound(p, pos, used);
  if (rest < 0) return;
  if (p.best_obj >= 0 && obj + rest >= p.best_obj) return;
  const int layer = p.order[pos];
  const int first = p.om[0][layer] <= p.om[1][layer] ? 0 : 1;
  for (int t = 0; t < 2; ++t) {
    const int c = t == 0 ? first : 1 - first;
    bool fits = true;
    for (int r = 0; r < kRes; ++r) {
      used[r] += p.rs[r][c][layer];
      if (p.active[r] && used[r] > p.limit[r]) fits = false;
    }
    if (fits) { p.cur[layer] = c; search(p, pos + 1, used, obj + p.om[c][layer]); }
    for (int r = 0; r < kRes; ++r) used[r] -= p.rs[r][c][layer];
  }
}

}  // namespace

extern "C" hq_status hq_ilp_solve(int32_t n_layers, const int64_t* omega, const int64_t* size, const int64_t* bops,
                                  const int64_t* latency, int64_t size_limit, int64_t bops_limit, int64_t latency_limit,
                                  int32_t* choice_out, int64_t* objective_out) {
  if (n_layers < 0 || n_layers > 4096 || !omega || !size || !bops || !latency || (n_layers > 0 && !choice_out))
    return HQ_ERR_INVALID_ARG;
  const int64_t* tabs[4] = {omega, size, bops, latency};
  for (int t = 0; t < 4; ++t)
    for (int i = 0; i < 2 * n_layers; ++i)
      if (tabs[t][i] < 0 || tabs[t][i] > kMaxValue) return HQ_ERR_INVALID_ARG;
  Problem p;
  p.n = n_layers;
  const int64_t limits[kRes] = {size_limit, bops_limit, latency_limit};
  for (int r = 0; r < kRes; ++r) { p.limit[r] = limits[r]; p.active[r] = limits[r] >= 0; }
  for (int c = 0; c < 2; ++c) {
    p.om[c].resize(n_layers);
    for (int r = 0; r < kRes; ++r) p.rs[r][c].resize(n_layers);
    for (int i = 0; i < n_layers; ++i) {
      p.om[c][i] = omega[2 * i + c];
      for (int r = 0; r < kRes; ++r) p.rs[r][c][i] = tabs[1 + r][2 * i + c];
    }
  }
  p.order.resize(n_layers);
  for (int i = 0; i < n_layers; ++i) p.order[i] = i;
  auto spread = [&](int i) { const int64_t d = p.om[0][i] - p.om[1][i]; return d < 0 ? -d : d; };
  std::stable_sort(p.order.begin(), p.order.end(), [&](int a, int b) { return spread(a) > spread(b); });
  p.pos_of.resize(n_layers);
  for (int k = 0; k < n_layers; ++k) p.pos_of[p.order[k]] = k;
  p.suf_min_om.assign(n_layers + 1, 0);
  for (int k = n_layers - 1; k >= 0; --k)
    p.suf_min_om[k] = p.suf_min_om[k + 1] + std::min(p.om[0][p.order[k]], p.om[1][p.order[k]]);
  for (int r = 0; r < kRes; ++r) {
    p.lo[r].resize(n_layers);
    for (int i = 0; i < n_layers; ++i) {
      const int64_t r0 = p.rs[r][0][i], r1 = p.rs[r][1][i];
      p.lo[r][i] = (r0 < r1 || (r0 == r1 && p.om[0][i] <= p.om[1][i])) ? 0 : 1;
    }
    p.suf_lo_om[r].assign(n_layers + 1, 0);
    p.suf_lo_rs[r].assign(n_layers + 1, 0);
    for (int k = n_layers - 1; k >= 0; --k) {
      const int i = p.order[k], l = p.lo[r][i];
      p.suf_lo_om[r][k] = p.suf_lo_om[r][k + 1] + p.om[l][i];
      p.suf_lo_rs[r][k] = p.suf_lo_rs[r][k + 1] + p.rs[r][l][i];
    }
    p.eff[r].resize(n_layers);
    for (int i = 0; i < n_layers; ++i) p.eff[r][i] = i;
    auto d_om = [&](int i) { const int l = p.lo[r][i]; return p.om[l][i] - p.om[1 - l][i]; };
    auto d_rs = [&](int i) { const int l = p.lo[r][i]; return p.rs[r][1 - l][i] - p.rs[r][l][i]; };
    std::stable_sort(p.eff[r].begin(), p.eff[r].end(), [&](int a, int b) {
      const int64_t oa = d_om(a), ob = d_om(b);
      if ((oa > 0) != (ob > 0)) return oa > 0;                    // upgrades that save something first
      if (oa <= 0) return false;
      // oa / ra > ob / rb, a cost of zero counting as the best ratio
      return (__int128)oa * d_rs(b) > (__int128)ob * d_rs(a);
    });
  }
  p.cur.assign(n_layers, 0);
  int64_t used[kRes] = {0, 0, 0};
  search(p, 0, used, 0);
  if (p.gave_up) return HQ_ERR_UNSUPPORTED;
  if (p.best_obj < 0) return HQ_ERR_INFEASIBLE;
  for (int i = 0; i < n_layers; ++i) choice_out[i] = p.best[i];
  if (objective_out) *objective_out = p.best_obj;
  return HQ_OK;
}
