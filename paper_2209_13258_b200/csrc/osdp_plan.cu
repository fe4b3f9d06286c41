// Execution-plan search on the host (Section 3.1 problem formulation and cost model, Algorithm 1; the
// per-slice planning of Section 3.3's last paragraph).  No device code: this file is part of the
// library so that the planner sits behind the same C ABI as the kernels whose measured times feed it.
//
// For one batch size the problem is a 0/1 knapsack.  Start from every operator in ZDP mode (least
// memory); switching operator i to DP costs w_i = M_i^(model) (1 - 1/N) more memory and saves one
// collective, c_i = (N-1)(alpha + S_i/N beta).  The search is the depth-first traversal with the paper's
// two prunings (memory above the limit; time not below the best plan so far), made tighter in two ways
// that do not change the optimum: operators are visited by decreasing saving per byte and the time
// pruning uses the fractional-knapsack bound of the unvisited rest; operators with identical (w, c)
// are decided as a group (how many of them run in DP), which removes the permutation symmetry of a
// transformer's repeated layers.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

#include "../../include/osdp.h"

namespace {

struct Op { double model, act, extra, S, gamma; };

inline double collective_cost(const Op &o, int world, double alpha, double beta) {
  return (double)(world - 1) * (alpha + o.S / (double)world * beta);
}

// Section 3.1, memory and time of a complete plan (summed in operator order).
void plan_cost(const Op *ops, int n, int world, double alpha, double beta, const uint8_t *modes, int b, double *mem,
               double *time) {
  double m = 0.0, t = 0.0;
  for (int i = 0; i < n; ++i) {
    const bool zdp = modes[i] != 0;
    m += (zdp ? ops[i].model / (double)world : ops[i].model) + (double)b * ops[i].act + ops[i].extra;
    t += (zdp ? 3.0 : 2.0) * collective_cost(ops[i], world, alpha, beta) + (double)b * ops[i].gamma;
  }
  *mem = m;
  *time = t;
}

struct Group {
  double w, c;            // memory cost and time saving of one member's switch to DP
  int first, count;       // members: order[first .. first + count)
};

struct Search {
  std::vector<Group> groups;
  std::vector<double> pw, pc;   // prefix sums of w and c over the members in visiting order
  std::vector<int> take, best_take;
  double best_saving;
  int64_t nodes, max_nodes;
  bool cut_short;

  // most that the members from position `pos` on can still save within `cap` (fractional relaxation)
  double bound(int pos, double cap) const {
    const int n = (int)pw.size() - 1;
    const double target = pw[pos] + cap;
    int j = (int)(std::upper_bound(pw.begin() + pos, pw.end(), target) - pw.begin()) - 1;   // pw[j] <= target
    if (j >= n) return pc[n] - pc[pos];
    const double wj = pw[j + 1] - pw[j];
    const double frac = wj > 0.0 ? (target - pw[j]) / wj : 1.0;
    return pc[j] - pc[pos] + frac * (pc[j + 1] - pc[j]);
  }

  void dfs(int g, double cap, double saving) {
    if (cut_short) return;
    if (++nodes > max_nodes) { cut_short = true; return; }
    if (g == (int)groups.size()) {
      if (saving > best_saving) { best_saving = saving; best_take = take; }
      return;
    }
    const Group &G = groups[g];
    // pruning 2: even the relaxed rest cannot beat the best plan so far
    if (saving + bound(G.first, cap) * (1.0 + 1e-12) <= best_saving) return;   // slack: prefix sums round
    int tmax = G.count;
    if (G.w > 0.0) {
      const double fit = std::floor(cap / G.w);
      if (fit < (double)tmax) tmax = (int)fit;      // pruning 1: more members in DP would exceed the memory limit
    }
    for (int t = tmax; t >= 0; --t) {
      take[g] = t;
      dfs(g + 1, cap - (double)t * G.w, saving + (double)t * G.c);
      if (cut_short) return;
    }
    take[g] = 0;
  }
};

// Best plan for one batch size.  Returns false if even all-ZDP exceeds the limit.
bool solve_batch(const Op *ops, int n, int world, double alpha, double beta, double limit, int b, int64_t max_nodes,
                 uint8_t *modes, double *time, int64_t *nodes, bool *cut_short) {
  std::vector<uint8_t> all_zdp((size_t)n, 1);
  double mem0, t0;
  plan_cost(ops, n, world, alpha, beta, all_zdp.data(), b, &mem0, &t0);
  if (!(mem0 <= limit)) return false;
  const double cap = limit - mem0;

  std::vector<int> order((size_t)n);
  std::vector<double> w((size_t)n), c((size_t)n);
  for (int i = 0; i < n; ++i) {
    order[i] = i;
    w[i] = ops[i].model * (1.0 - 1.0 / (double)world);
    c[i] = collective_cost(ops[i], world, alpha, beta);
  }
  auto density_before = [&](int a, int bb) {   // a's saving per byte above b's; free savings first
    const double l = c[a] * w[bb], r = c[bb] * w[a];
    if (l != r) return l > r;
    if (w[a] != w[bb]) return w[a] < w[bb];
    if (c[a] != c[bb]) return c[a] > c[bb];
    return a < bb;
  };
  std::sort(order.begin(), order.end(), density_before);

  Search S;
  S.pw.assign((size_t)n + 1, 0.0);
  S.pc.assign((size_t)n + 1, 0.0);
  for (int j = 0; j < n; ++j) {
    const int i = order[j];
    S.pw[j + 1] = S.pw[j] + w[i];
    S.pc[j + 1] = S.pc[j] + c[i];
    if (!S.groups.empty() && S.groups.back().w == w[i] && S.groups.back().c == c[i]) ++S.groups.back().count;
    else S.groups.push_back(Group{w[i], c[i], j, 1});
  }
  S.take.assign(S.groups.size(), 0);
  S.best_take.assign(S.groups.size(), 0);
  S.best_saving = -1.0;
  S.nodes = 0;
  S.max_nodes = max_nodes;
  S.cut_short = false;
  S.dfs(0, cap, 0.0);
  *nodes += S.nodes;
  *cut_short = S.cut_short;

  std::memset(modes, 1, (size_t)n);
  for (size_t g = 0; g < S.groups.size(); ++g)
    for (int t = 0; t < S.best_take[g]; ++t) modes[order[S.groups[g].first + t]] = 0;
  double mem;
  plan_cost(ops, n, world, alpha, beta, modes, b, &mem, time);
  // Rounding guard: the search adds savings, the verdict adds the paper's sums; if the two disagree on
  // the last bit at the limit, give up the cheapest saving until the plan fits as the verdict counts.
  while (mem > limit) {
    int drop = -1;
    for (int i = 0; i < n; ++i)
      if (modes[i] == 0 && w[i] > 0.0 && (drop < 0 || c[i] < c[drop])) drop = i;
    if (drop < 0) break;
    modes[drop] = 1;
    plan_cost(ops, n, world, alpha, beta, modes, b, &mem, time);
  }
  return true;
}

int check_inputs(const double *ops, int n, int world, double alpha, double beta) {
  if (!ops) return OSDP_ERR_NULL_POINTER;
  if (n < 1 || n > 16384 || world < 1) return OSDP_ERR_BAD_SHAPE;
  if (!(alpha >= 0.0) || !(beta >= 0.0) || !std::isfinite(alpha) || !std::isfinite(beta)) return OSDP_ERR_BAD_SHAPE;
  for (int i = 0; i < 5 * n; ++i)
    if (!(ops[i] >= 0.0) || !std::isfinite(ops[i])) return OSDP_ERR_BAD_SHAPE;
  return OSDP_OK;
}

}  // namespace

extern "C" {

int osdp_plan_cost(const double *ops, int n, int world, double alpha, double beta, const uint8_t *modes, int batch,
                   double *memory, double *time) {
  int rc = check_inputs(ops, n, world, alpha, beta);
  if (rc) return rc;
  if (!modes || !memory || !time) return OSDP_ERR_NULL_POINTER;
  if (batch < 1) return OSDP_ERR_BAD_SHAPE;
  plan_cost(reinterpret_cast<const Op *>(ops), n, world, alpha, beta, modes, batch, memory, time);
  return OSDP_OK;
}

int osdp_plan_search(const double *ops, int n, int world, double alpha, double beta, double mem_limit,
                     int max_batch, int64_t max_nodes, uint8_t *modes, int *batch, double *time_per_sample,
                     int64_t *nodes_visited) {
  int rc = check_inputs(ops, n, world, alpha, beta);
  if (rc) return rc;
  if (!modes || !batch || !time_per_sample) return OSDP_ERR_NULL_POINTER;
  if (max_batch < 1 || !(mem_limit >= 0.0)) return OSDP_ERR_BAD_SHAPE;
  if (max_nodes <= 0) max_nodes = (int64_t)200 * 1000 * 1000;
  const Op *o = reinterpret_cast<const Op *>(ops);
  std::vector<uint8_t> cur((size_t)n);
  double best = std::numeric_limits<double>::infinity();
  int best_b = 0;
  int64_t nodes = 0;
  bool any_cut = false;
  for (int b = 1; b <= max_batch; ++b) {          // Algorithm 1: grow the batch until nothing fits
    double t = 0.0;
    bool cut = false;
    if (!solve_batch(o, n, world, alpha, beta, mem_limit, b, max_nodes, cur.data(), &t, &nodes, &cut)) break;
    any_cut = any_cut || cut;
    const double per_sample = t / (double)b;
    if (per_sample < best) {                      // the scheduler keeps the candidate of highest throughput
      best = per_sample;
      best_b = b;
      std::memcpy(modes, cur.data(), (size_t)n);
    }
  }
  *batch = best_b;
  *time_per_sample = best;
  if (nodes_visited) *nodes_visited = nodes;
  return any_cut ? OSDP_ERR_SEARCH_LIMIT : OSDP_OK;
}

int osdp_plan_expand_slices(const double *op, int k, double overhead, double *slices) {
  if (!op || !slices) return OSDP_ERR_NULL_POINTER;
  if (k < 1 || k > OSDP_MAX_SPLIT) return OSDP_ERR_BAD_SPLIT;
  if (!(overhead > -1.0) || !std::isfinite(overhead)) return OSDP_ERR_BAD_SHAPE;
  for (int s = 0; s < k; ++s) {
    for (int j = 0; j < 4; ++j) slices[5 * s + j] = op[j] / (double)k;
    slices[5 * s + 4] = op[4] * (1.0 + overhead) / (double)k;
  }
  return OSDP_OK;
}

}  // extern "C"
