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


// ---- granularity left free: every operator picks one of its allowed granularities and how many of its
// slices run in DP (Section 3.3, last paragraph).  For one batch size this is a multiple-choice knapsack:
// one option (k, j) per operator, least total time within the memory limit.

struct Option { double mem, time; int k, dp; };

// Memory and time of an operator cut k ways with its first j slices in DP, summed slice by slice.
void sliced_cost(const Op &o, int k, double overhead, int j, int world, double alpha, double beta, int b, double *mem,
                 double *time) {
  const Op s{o.model / (double)k, o.act / (double)k, o.extra / (double)k, o.S / (double)k,
             o.gamma * (1.0 + overhead) / (double)k};
  double m = 0.0, t = 0.0;
  for (int i = 0; i < k; ++i) {
    const bool zdp = i >= j;
    m += (zdp ? s.model / (double)world : s.model) + (double)b * s.act + s.extra;
    t += (zdp ? 3.0 : 2.0) * collective_cost(s, world, alpha, beta) + (double)b * s.gamma;
  }
  *mem = m;
  *time = t;
}

struct Choice {
  std::vector<Option> opts;   // undominated, memory ascending, time strictly descending
  std::vector<int> hull;      // indices into opts: lower convex hull, for the relaxation
};

struct Segment { double dm, dt; int pos; };   // one hull step of the operator at visiting position pos

struct GranSearch {
  std::vector<const Choice *> ch;        // per visiting position
  std::vector<char> same_as_prev;        // identical operator at pos - 1: options in non-decreasing index order
  std::vector<double> min_mem, min_time; // suffix sums over the least-memory options
  std::vector<Segment> segs;             // all hull steps, steepest time saving per byte first
  std::vector<int> pick, best_pick;
  double best;
  int64_t nodes, max_nodes;
  bool cut_short;

  // least time of positions pos.. within cap if options could be mixed fractionally; +inf if nothing fits
  double bound(int pos, double cap) const {
    if (min_mem[pos] > cap) return std::numeric_limits<double>::infinity();
    double room = cap - min_mem[pos], t = min_time[pos];
    for (const Segment &g : segs) {
      if (g.pos < pos) continue;
      if (g.dm <= room) { room -= g.dm; t += g.dt; }
      else { t += g.dt * (room / g.dm); break; }
    }
    return t;
  }

  void dfs(int pos, double cap, double t) {
    if (cut_short) return;
    if (++nodes > max_nodes) { cut_short = true; return; }
    const int n = (int)ch.size();
    if (pos == n) {
      if (t < best) { best = t; best_pick = pick; }
      return;
    }
    const double lb = t + bound(pos, cap);
    if (!(lb * (1.0 - 1e-12) < best)) return;                      // pruning 2 (time), relaxed
    const std::vector<Option> &o = ch[pos]->opts;
    const int lo = same_as_prev[pos] ? pick[pos - 1] : 0;
    for (int i = (int)o.size() - 1; i >= lo; --i) {                // fastest (largest) option first
      if (o[i].mem + min_mem[pos + 1] > cap) continue;             // pruning 1 (memory)
      pick[pos] = i;
      dfs(pos + 1, cap - o[i].mem, t + o[i].time);
      if (cut_short) return;
    }
  }
};

// Options of one operator whose gathered slice, if any slice is in ZDP, is at most `tau` bytes.
void build_choice(const Op &op, const int *ks, const double *ovh, int ncand, int world, double alpha, double beta, int b,
                  double tau, Choice *c) {
  std::vector<Option> all;
  for (int a = 0; a < ncand; ++a)
    for (int j = 0; j <= ks[a]; ++j) {
      if (j < ks[a] && op.S / (double)ks[a] > tau) continue;
      Option o{0.0, 0.0, ks[a], j};
      sliced_cost(op, ks[a], ovh[a], j, world, alpha, beta, b, &o.mem, &o.time);
      all.push_back(o);
    }
  std::stable_sort(all.begin(), all.end(), [](const Option &x, const Option &y) {
    return x.mem != y.mem ? x.mem < y.mem : x.time < y.time;
  });
  c->opts.clear();
  for (const Option &o : all)
    if (c->opts.empty() || o.time < c->opts.back().time) {
      if (!c->opts.empty() && o.mem == c->opts.back().mem) continue;
      c->opts.push_back(o);
    }
  c->hull.clear();
  for (int i = 0; i < (int)c->opts.size(); ++i) {
    while (c->hull.size() >= 2) {
      const Option &p = c->opts[c->hull[c->hull.size() - 2]], &q = c->opts[c->hull.back()], &r = c->opts[i];
      // q lies on or above the chord p-r: drop it
      if ((q.time - p.time) * (r.mem - p.mem) >= (r.time - p.time) * (q.mem - p.mem)) c->hull.pop_back();
      else break;
    }
    c->hull.push_back(i);
  }
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

int osdp_plan_search_granularity(const double *ops, int n, const int *cand_begin, const int *cand_k,
                                 const double *cand_overhead, int world, double alpha, double beta, double mem_limit,
                                 double surge_factor, int max_batch, int64_t max_nodes, int *k_out, int *dp_slices,
                                 int *batch, double *time_per_sample, int64_t *nodes_visited) {
  int rc = check_inputs(ops, n, world, alpha, beta);
  if (rc) return rc;
  if (!cand_begin || !cand_k || !cand_overhead || !k_out || !dp_slices || !batch || !time_per_sample)
    return OSDP_ERR_NULL_POINTER;
  if (max_batch < 1 || !(mem_limit >= 0.0) || cand_begin[0] != 0) return OSDP_ERR_BAD_SHAPE;
  if (!(surge_factor >= 0.0) || !std::isfinite(surge_factor)) return OSDP_ERR_BAD_SHAPE;
  for (int i = 0; i < n; ++i) {
    if (cand_begin[i + 1] <= cand_begin[i]) return OSDP_ERR_BAD_SHAPE;     // every operator needs a candidate
    for (int a = cand_begin[i]; a < cand_begin[i + 1]; ++a) {
      if (cand_k[a] < 1 || cand_k[a] > OSDP_MAX_SPLIT) return OSDP_ERR_BAD_SPLIT;
      if (!(cand_overhead[a] > -1.0) || !std::isfinite(cand_overhead[a])) return OSDP_ERR_BAD_SHAPE;
    }
  }
  if (max_nodes <= 0) max_nodes = (int64_t)200 * 1000 * 1000;
  const Op *o = reinterpret_cast<const Op *>(ops);

  // visiting order: identical operators (same five figures, same candidates) next to each other
  auto same = [&](int a, int b) {
    if (std::memcmp(&o[a], &o[b], sizeof(Op)) != 0) return false;
    const int na = cand_begin[a + 1] - cand_begin[a];
    if (na != cand_begin[b + 1] - cand_begin[b]) return false;
    for (int j = 0; j < na; ++j)
      if (cand_k[cand_begin[a] + j] != cand_k[cand_begin[b] + j] ||
          cand_overhead[cand_begin[a] + j] != cand_overhead[cand_begin[b] + j]) return false;
    return true;
  };
  std::vector<int> cls((size_t)n), reps;             // class of each operator, representative of each class
  for (int i = 0; i < n; ++i) {
    int c = -1;
    for (size_t r = 0; r < reps.size() && c < 0; ++r)
      if (same(i, reps[r])) c = (int)r;
    if (c < 0) { c = (int)reps.size(); reps.push_back(i); }
    cls[i] = c;
  }
  std::vector<int> order((size_t)n);
  for (int i = 0; i < n; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cls[a] < cls[b]; });

  // The gathered slice of a ZDP operator is transient memory on top of the sums of Section 3.1: the largest
  // one, times surge_factor, counts against the limit.  A maximum does not fit a knapsack, so the search
  // runs once per possible value tau of that maximum, with only the options whose gathered slice is at
  // most tau and with the limit lowered by surge_factor * tau; the best over all tau is the optimum.
  std::vector<double> taus;
  if (surge_factor > 0.0) {
    taus.push_back(0.0);
    for (int i = 0; i < n; ++i)
      for (int a = cand_begin[i]; a < cand_begin[i + 1]; ++a) taus.push_back(o[i].S / (double)cand_k[a]);
    std::sort(taus.begin(), taus.end());
    taus.erase(std::unique(taus.begin(), taus.end()), taus.end());
  } else {
    taus.push_back(std::numeric_limits<double>::infinity());
  }

  double best = std::numeric_limits<double>::infinity();
  int best_b = 0;
  int64_t nodes = 0;
  bool any_cut = false;
  std::vector<Choice> choice(reps.size());
  for (int b = 1; b <= max_batch; ++b) {             // Algorithm 1: grow the batch until nothing fits
    double best_t = std::numeric_limits<double>::infinity();   // least time at this batch size, over all tau
    int64_t nodes_b = 0;
    std::vector<int> best_k((size_t)n), best_dp((size_t)n);
    for (double tau : taus) {
      const double cap = surge_factor > 0.0 ? mem_limit - surge_factor * tau : mem_limit;
      if (!(cap >= 0.0)) break;
      for (size_t r = 0; r < reps.size(); ++r) {
        const int i = reps[r];
        build_choice(o[i], cand_k + cand_begin[i], cand_overhead + cand_begin[i], cand_begin[i + 1] - cand_begin[i],
                     world, alpha, beta, b, tau, &choice[r]);
      }
      GranSearch S;
      S.ch.resize((size_t)n);
      S.same_as_prev.assign((size_t)n, 0);
      S.min_mem.assign((size_t)n + 1, 0.0);
      S.min_time.assign((size_t)n + 1, 0.0);
      for (int p = 0; p < n; ++p) {
        S.ch[p] = &choice[cls[order[p]]];
        S.same_as_prev[p] = p > 0 && cls[order[p]] == cls[order[p - 1]];
        const Choice &c = *S.ch[p];
        for (size_t h = 1; h < c.hull.size(); ++h)
          S.segs.push_back(Segment{c.opts[c.hull[h]].mem - c.opts[c.hull[h - 1]].mem,
                                   c.opts[c.hull[h]].time - c.opts[c.hull[h - 1]].time, p});
      }
      for (int p = n - 1; p >= 0; --p) {
        S.min_mem[p] = S.min_mem[p + 1] + S.ch[p]->opts.front().mem;
        S.min_time[p] = S.min_time[p + 1] + S.ch[p]->opts.front().time;
      }
      if (S.min_mem[0] > cap) continue;
      std::stable_sort(S.segs.begin(), S.segs.end(),
                       [](const Segment &x, const Segment &y) { return x.dt * y.dm < y.dt * x.dm; });
      S.pick.assign((size_t)n, 0);
      S.best_pick.assign((size_t)n, 0);
      S.best = best_t;                               // only plans faster than the best of the earlier tau matter
      {
        // first plan: from the least-memory options, hull steps by decreasing time saved per byte while they fit
        // (the relaxation's solution without its fractional step); it makes the time pruning bite at once
        std::vector<int> h((size_t)n, 0);
        std::vector<char> stuck((size_t)n, 0);
        double room = cap - S.min_mem[0], t = S.min_time[0];
        for (const Segment &g : S.segs) {
          if (stuck[g.pos]) continue;
          if (g.dm <= room) { room -= g.dm; t += g.dt; ++h[g.pos]; }
          else stuck[g.pos] = 1;                       // an operator's steps come in order: skip its later ones
        }
        if (t < S.best) {
          S.best = t;
          for (int p = 0; p < n; ++p) S.best_pick[p] = S.ch[p]->hull[h[p]];
        }
      }
      S.nodes = 0;
      S.max_nodes = std::max<int64_t>(1, max_nodes - nodes_b);   // one node budget per batch size
      S.cut_short = false;
      S.dfs(0, cap, 0.0);
      nodes += S.nodes;
      nodes_b += S.nodes;
      any_cut = any_cut || S.cut_short;
      if (!(S.best < best_t)) {
        // nothing faster under this tau; if no plan is known yet because the budget ran out before the
        // first leaf, take the least-memory options (best_pick all zero), which fit
        if (best_t < std::numeric_limits<double>::infinity() || !S.cut_short) continue;
      }
      // verdict in the caller's operator order, summed the way a plan is priced; if the last bit of the
      // memory sum lands above the limit, fall back to least-memory options one operator at a time
      std::vector<int> pick((size_t)n);
      for (int p = 0; p < n; ++p) pick[order[p]] = S.best_pick[p];
      double mem = 0.0, t = 0.0;
      auto price = [&]() {
        mem = 0.0; t = 0.0;
        for (int i = 0; i < n; ++i) { const Option &q = choice[cls[i]].opts[pick[i]]; mem += q.mem; t += q.time; }
      };
      price();
      for (int i = n - 1; i >= 0 && mem > cap; --i)
        if (pick[i] != 0) { pick[i] = 0; price(); }
      if (mem > cap) continue;
      if (t < best_t) {
        best_t = t;
        for (int i = 0; i < n; ++i) { const Option &q = choice[cls[i]].opts[pick[i]]; best_k[i] = q.k; best_dp[i] = q.dp; }
      }
    }
    if (!(best_t < std::numeric_limits<double>::infinity())) break;
    const double per_sample = best_t / (double)b;
    if (per_sample < best) {
      best = per_sample;
      best_b = b;
      for (int i = 0; i < n; ++i) { k_out[i] = best_k[i]; dp_slices[i] = best_dp[i]; }
    }
  }
  *batch = best_b;
  *time_per_sample = best;
  if (nodes_visited) *nodes_visited = nodes;
  return any_cut ? OSDP_ERR_SEARCH_LIMIT : OSDP_OK;
}

}  // extern "C"
