// Threshold assignment of the offline calibration: one candidate per head under a global sparsity
// budget (section "Error-guided Budgeted Calibration": minimise the summed measured errors subject to
// one choice per head and a mean realised sparsity of at least S_min; last step of Algorithm 2).
//
// This is an offline problem on a few thousand numbers (heads x candidates), so it runs on the host:
// an exact multiple-choice-knapsack solver, no kernel.  Method: dynamic programming over the heads in
// index order.  A state is a pair (sparsity so far, error so far); after each head the states that
// another state beats on both counts are dropped, and so are the states that cannot win any more --
// their error plus a lower bound on what the remaining heads must still cost (the linear relaxation
// of the rest: cheapest error per unit of sparsity first) is no better than a solution already in
// hand.  The first solution in hand comes from rounding the relaxation of the whole problem up.
// Both running sums are accumulated head by head in index order, so the feasibility test and the
// objective of the answer are the plain left-to-right sums of its choices.
#include <math.h>

#include <algorithm>
#include <limits>
#include <vector>

#include "heart.h"

namespace {

struct Cand {
  double s, e;
  int k;  // the caller's candidate index
};

struct Inc {  // one step along a head's lower convex hull: from hull point `pos - 1` to `pos`
  double ds, de, slope;
  int cls, pos;
};

struct State {
  double s, e;
  int parent;  // index into the previous head's state list
  int cand;    // frontier index chosen for this head
};

constexpr size_t kStateLimit = 40u * 1000u * 1000u;  // total states kept; beyond it the search stops early

struct Problem {
  int M, K;
  const double *E, *S;
  double S_min;
  std::vector<std::vector<Cand>> frontier;  // per head: non-dominated candidates, s and e ascending
  std::vector<std::vector<int>> hull;       // per head: frontier indices on the lower convex hull
};

// mean sparsity and objective of an assignment, as plain left-to-right sums over the heads
void evaluate(const Problem &p, const std::vector<int> &choice, double *mean_s, double *obj) {
  double e = 0.0, s = 0.0;
  for (int i = 0; i < p.M; ++i) {
    e += p.E[(size_t)i * p.K + choice[i]];
    s += p.S[(size_t)i * p.K + choice[i]];
  }
  *mean_s = s / (double)p.M;
  *obj = e;
}

void build_frontiers(Problem &p) {
  p.frontier.assign(p.M, {});
  p.hull.assign(p.M, {});
  for (int i = 0; i < p.M; ++i) {
    std::vector<Cand> c(p.K);
    for (int k = 0; k < p.K; ++k) c[k] = {p.S[(size_t)i * p.K + k], p.E[(size_t)i * p.K + k], k};
    // most sparsity first; among equal sparsity the smaller error, then the smaller index
    std::sort(c.begin(), c.end(), [](const Cand &a, const Cand &b) {
      if (a.s != b.s) return a.s > b.s;
      if (a.e != b.e) return a.e < b.e;
      return a.k < b.k;
    });
    std::vector<Cand> f;
    double best_e = std::numeric_limits<double>::infinity();
    for (const Cand &x : c)  // kept only if strictly cheaper than everything at least as sparse
      if (x.e < best_e) {
        f.push_back(x);
        best_e = x.e;
      }
    std::reverse(f.begin(), f.end());  // s ascending, e ascending; f[0] is the head's cheapest candidate
    p.frontier[i] = f;
    std::vector<int> &h = p.hull[i];
    for (int j = 0; j < (int)f.size(); ++j) {
      while (h.size() >= 2) {
        const Cand &a = f[h[h.size() - 2]], &b = f[h.back()];
        // b lies on or above the segment a -> f[j]: not on the lower hull
        if ((b.e - a.e) * (f[j].s - a.s) >= (f[j].e - a.e) * (b.s - a.s))
          h.pop_back();
        else
          break;
      }
      h.push_back(j);
    }
  }
}

// The remaining heads' hull steps, cheapest error per unit of sparsity first, with running totals.
struct Relaxation {
  std::vector<Inc> inc;
  std::vector<double> cum_s, cum_e;
  void rebuild_totals() {
    cum_s.resize(inc.size());
    cum_e.resize(inc.size());
    double s = 0.0, e = 0.0;
    for (size_t n = 0; n < inc.size(); ++n) {
      s += inc[n].ds;
      e += inc[n].de;
      cum_s[n] = s;
      cum_e[n] = e;
    }
  }
  void drop_class(int cls) {
    inc.erase(std::remove_if(inc.begin(), inc.end(), [cls](const Inc &x) { return x.cls == cls; }), inc.end());
    rebuild_totals();
  }
  // least extra error with which the remaining heads can add `t` of sparsity to their cheapest choices
  double cost(double t) const {
    if (!(t > 0.0)) return 0.0;
    const size_t n = std::lower_bound(cum_s.begin(), cum_s.end(), t) - cum_s.begin();
    if (n == cum_s.size()) return std::numeric_limits<double>::infinity();
    const double s0 = n ? cum_s[n - 1] : 0.0, e0 = n ? cum_e[n - 1] : 0.0;
    return e0 + (t - s0) * inc[n].slope;
  }
};

}  // namespace

extern "C" int heart_assign_thresholds(const double *E, const double *S, int32_t n_heads, int32_t n_candidates,
                                       double S_min, int32_t *choice_out, double *objective_out,
                                       double *mean_sparsity_out, int32_t *proved_optimal_out) {
  if (!E || !S || !choice_out || n_heads <= 0 || n_candidates <= 0 || isnan(S_min)) return HEART_ERR_INVALID;
  Problem p;
  p.M = n_heads;
  p.K = n_candidates;
  p.E = E;
  p.S = S;
  p.S_min = S_min;
  for (size_t n = 0; n < (size_t)p.M * p.K; ++n)
    if (!isfinite(E[n]) || !isfinite(S[n])) return HEART_ERR_INVALID;
  build_frontiers(p);
  const int M = p.M;
  const double T = S_min * (double)M;  // the budget as a sum (bounds only; the exact test is evaluate())

  std::vector<int> best(M), trial(M);
  double best_obj = std::numeric_limits<double>::infinity(), best_mean = 0.0;
  auto consider = [&](const std::vector<int> &choice) {
    double ms, obj;
    evaluate(p, choice, &ms, &obj);
    if (ms >= S_min && obj < best_obj) {
      best = choice;
      best_obj = obj;
      best_mean = ms;
    }
  };
  // (1) every head at its sparsest candidate: the largest mean any assignment reaches
  for (int i = 0; i < M; ++i) trial[i] = p.frontier[i].back().k;
  consider(trial);
  if (!(best_obj < std::numeric_limits<double>::infinity())) return HEART_ERR_INFEASIBLE;
  // (2) every head at its cheapest candidate: optimal whenever it meets the budget
  for (int i = 0; i < M; ++i) trial[i] = p.frontier[i][0].k;
  {
    double ms, obj;
    evaluate(p, trial, &ms, &obj);
    if (ms >= S_min) {
      for (int i = 0; i < M; ++i) choice_out[i] = trial[i];
      if (objective_out) *objective_out = obj;
      if (mean_sparsity_out) *mean_sparsity_out = ms;
      if (proved_optimal_out) *proved_optimal_out = 1;
      return HEART_OK;
    }
  }
  // (3) the relaxation of the whole problem, rounded up, as the first solution to beat
  Relaxation rel;
  std::vector<double> base_s_suffix(M + 1, 0.0), base_e_suffix(M + 1, 0.0), max_s_suffix(M + 1, 0.0);
  for (int i = M - 1; i >= 0; --i) {
    base_s_suffix[i] = base_s_suffix[i + 1] + p.frontier[i][0].s;
    base_e_suffix[i] = base_e_suffix[i + 1] + p.frontier[i][0].e;
    max_s_suffix[i] = max_s_suffix[i + 1] + p.frontier[i].back().s;
  }
  for (int i = 0; i < M; ++i)
    for (size_t h = 1; h < p.hull[i].size(); ++h) {
      const Cand &a = p.frontier[i][p.hull[i][h - 1]], &b = p.frontier[i][p.hull[i][h]];
      rel.inc.push_back({b.s - a.s, b.e - a.e, (b.e - a.e) / (b.s - a.s), i, (int)h});
    }
  std::sort(rel.inc.begin(), rel.inc.end(), [](const Inc &a, const Inc &b) {
    if (a.slope != b.slope) return a.slope < b.slope;
    if (a.cls != b.cls) return a.cls < b.cls;
    return a.pos < b.pos;
  });
  rel.rebuild_totals();
  {
    std::vector<int> pos(M, 0);
    double need = T - base_s_suffix[0], got = 0.0;
    for (const Inc &x : rel.inc) {
      if (got >= need) break;
      pos[x.cls] = std::max(pos[x.cls], x.pos);
      got += x.ds;
    }
    for (int i = 0; i < M; ++i) trial[i] = p.frontier[i][p.hull[i][pos[i]]].k;
    consider(trial);
    // rounding of the sums may leave it a hair short: one more step of the cheapest kind, if so
    for (const Inc &x : rel.inc) {
      double ms, obj;
      evaluate(p, trial, &ms, &obj);
      if (ms >= S_min) break;
      if (x.pos > pos[x.cls]) {
        pos[x.cls] = x.pos;
        trial[x.cls] = p.frontier[x.cls][p.hull[x.cls][x.pos]].k;
      }
    }
    consider(trial);
  }
  // (4) dynamic programming over the heads with dominance and bound pruning
  const double feas_slack = 1e-9 * (fabs(T) + max_s_suffix[0] + 1.0);
  std::vector<std::vector<State>> stage(M);
  std::vector<State> merged;
  size_t total_states = 0;
  bool complete = true;
  for (int i = 0; i < M && complete; ++i) {
    rel.drop_class(i);  // the relaxation now covers heads i+1 .. M-1
    const std::vector<Cand> &f = p.frontier[i];
    const std::vector<State> *prev = i ? &stage[i - 1] : nullptr;
    const size_t n_prev = prev ? prev->size() : 1;
    merged.clear();
    merged.reserve(n_prev * f.size());
    for (size_t n = 0; n < n_prev; ++n) {
      const double s0 = prev ? (*prev)[n].s : 0.0, e0 = prev ? (*prev)[n].e : 0.0;
      for (int j = 0; j < (int)f.size(); ++j) {
        const double s = s0 + f[j].s, e = e0 + f[j].e;  // head-by-head sums in index order
        // cannot reach the budget any more, even with every remaining head at its sparsest
        if (s + max_s_suffix[i + 1] < T - feas_slack) continue;
        // cannot beat the solution in hand: error so far + the rest at their cheapest + the cheapest way
        // to buy the missing sparsity
        const double bound = e + base_e_suffix[i + 1] + rel.cost(T - feas_slack - s - base_s_suffix[i + 1]);
        const double slack = 1e-11 * (fabs(bound) + fabs(best_obj)) + std::numeric_limits<double>::min();
        if (!(bound - slack < best_obj)) continue;
        merged.push_back({s, e, (int)n, j});
      }
    }
    // dominance: sparsest first, keep a state only if it is strictly cheaper than all sparser ones
    std::sort(merged.begin(), merged.end(), [](const State &a, const State &b) {
      if (a.s != b.s) return a.s > b.s;
      return a.e < b.e;
    });
    std::vector<State> &out = stage[i];
    double cheapest = std::numeric_limits<double>::infinity();
    for (const State &x : merged)
      if (x.e < cheapest) {
        out.push_back(x);
        cheapest = x.e;
      }
    total_states += out.size();
    if (total_states > kStateLimit) complete = false;
    if (out.empty()) break;  // nothing can beat the solution in hand
  }
  if (complete && !stage[M - 1].empty()) {
    // the final states carry the exact left-to-right sums of their assignments
    int win = -1;
    double win_e = best_obj;
    const std::vector<State> &last = stage[M - 1];
    for (size_t n = 0; n < last.size(); ++n)
      if (last[n].s / (double)M >= S_min && last[n].e < win_e) {
        win = (int)n;
        win_e = last[n].e;
      }
    if (win >= 0) {
      int at = win;
      for (int i = M - 1; i >= 0; --i) {
        const State &x = stage[i][at];
        trial[i] = p.frontier[i][x.cand].k;
        at = x.parent;
      }
      consider(trial);
    }
  }
  for (int i = 0; i < M; ++i) choice_out[i] = best[i];
  if (objective_out) *objective_out = best_obj;
  if (mean_sparsity_out) *mean_sparsity_out = best_mean;
  if (proved_optimal_out) *proved_optimal_out = complete ? 1 : 0;
  return HEART_OK;
}
