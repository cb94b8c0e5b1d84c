// Round scheduler (CPU): deadline-aware allocation and the group-knapsack DP of Algorithm 1.
#include <cmath>
#include <limits>
#include <vector>

#include "../../include/dit_sched.h"

extern "C" dit_status dit_sched_allocate(const int32_t* gpus, const double* step_time, int32_t n_degrees, int32_t steps,
                                         double time_budget, dit_sched_option* out, int32_t* n_out, double* gpu_time,
                                         int32_t* feasible) {
  if (!gpus || !step_time || !out || !n_out || !gpu_time || !feasible || n_degrees < 1 || steps < 0) return DIT_ERR_INVALID_ARG;
  for (int d = 0; d < n_degrees; ++d)
    if (gpus[d] < 1 || !(step_time[d] > 0.0)) return DIT_ERR_INVALID_ARG;
  double best_cost = std::numeric_limits<double>::infinity(), best_time = 0.0;
  int best_a = -1, best_b = -1, best_na = 0;
  // every pair of degrees (a <= b in table order) and every split of the steps between them
  for (int a = 0; a < n_degrees; ++a) {
    for (int b = a; b < n_degrees; ++b) {
      for (int na = (a == b ? steps : 0); na <= steps; ++na) {
        const int nb = steps - na;
        const double t = na * step_time[a] + nb * step_time[b];
        if (t > time_budget) continue;
        const double cost = na * (gpus[a] * step_time[a]) + nb * (gpus[b] * step_time[b]);
        if (cost < best_cost || (cost == best_cost && t < best_time)) {
          best_cost = cost; best_time = t; best_a = a; best_b = b; best_na = na;
        }
      }
    }
  }
  if (best_a < 0) {   // infeasible: everything at the fastest degree
    int f = 0;
    for (int d = 1; d < n_degrees; ++d)
      if (step_time[d] < step_time[f]) f = d;
    out[0] = dit_sched_option{steps, gpus[f], step_time[f]};
    *n_out = 1;
    *gpu_time = steps * (gpus[f] * step_time[f]);
    *feasible = 0;
    return DIT_OK;
  }
  int n = 0;
  if (best_na > 0 || steps == 0) out[n++] = dit_sched_option{best_na, gpus[best_a], step_time[best_a]};
  if (steps - best_na > 0 && best_b != best_a) out[n++] = dit_sched_option{steps - best_na, gpus[best_b], step_time[best_b]};
  *n_out = n;
  *gpu_time = best_cost;
  *feasible = 1;
  return DIT_OK;
}

extern "C" dit_status dit_sched_round(const dit_sched_request* reqs, int32_t n_requests, int32_t n_gpus, double tau,
                                      double t_now, int32_t* chosen, int32_t* steps_done, int32_t* n_survivors,
                                      int32_t* gpus_used) {
  if (n_requests < 0 || n_gpus < 0 || !(tau > 0.0) || (n_requests > 0 && (!reqs || !chosen))) return DIT_ERR_INVALID_ARG;
  for (int i = 0; i < n_requests; ++i) {
    if (reqs[i].n_options < 0 || (reqs[i].n_options > 0 && !reqs[i].options) || !(reqs[i].t_min > 0.0)) return DIT_ERR_INVALID_ARG;
    for (int m = 0; m < reqs[i].n_options; ++m)
      if (reqs[i].options[m].steps < 0 || reqs[i].options[m].gpus < 1 || !(reqs[i].options[m].step_time > 0.0))
        return DIT_ERR_INVALID_ARG;
  }
  const double t_next = t_now + tau;
  const int N = n_gpus;
  // per request: candidate options (index -1 = none), their width, progress and survival flag
  struct Cand { int option, width, q, survives; };
  std::vector<std::vector<Cand>> cands(n_requests);
  for (int i = 0; i < n_requests; ++i) {
    const dit_sched_request& r = reqs[i];
    long long total = 0;
    for (int m = 0; m < r.n_options; ++m) total += r.options[m].steps;
    auto survives = [&](long long remaining) { return t_next + static_cast<double>(remaining) * r.t_min <= r.deadline ? 1 : 0; };
    cands[i].push_back(Cand{-1, 0, 0, survives(total)});
    for (int m = 0; m < r.n_options; ++m) {
      const dit_sched_option& o = r.options[m];
      const double fit = std::floor(tau / o.step_time);
      const int q = static_cast<int>(std::min<double>(o.steps, fit));
      if (q <= 0 || o.gpus > N) continue;
      cands[i].push_back(Cand{m, o.gpus, q, survives(total - q)});
    }
  }
  // dp[c]: best (survivors, steps completed this round), compared in that order, among the requests
  // processed so far with exactly c GPUs in use; packed as survivors * 2^32 + steps
  const long long kNegInf = std::numeric_limits<long long>::min() / 2;
  std::vector<long long> dp(N + 1, kNegInf), next(N + 1);
  dp[0] = 0;
  std::vector<std::vector<int>> pick(n_requests, std::vector<int>(N + 1, -1));   // back-pointers: candidate index
  for (int i = 0; i < n_requests; ++i) {
    for (int c = 0; c <= N; ++c) {
      long long best = kNegInf;
      int arg = -1;
      for (size_t k = 0; k < cands[i].size(); ++k) {
        const Cand& o = cands[i][k];
        if (o.width > c || dp[c - o.width] == kNegInf) continue;
        const long long v = dp[c - o.width] + (static_cast<long long>(o.survives) << 32) + o.q;
        if (v > best) { best = v; arg = static_cast<int>(k); }
      }
      next[c] = best;
      pick[i][c] = arg;
    }
    dp.swap(next);
  }
  int c_star = 0;
  for (int c = 1; c <= N; ++c)
    if (dp[c] > dp[c_star]) c_star = c;
  if (n_survivors) *n_survivors = dp[c_star] == kNegInf ? 0 : static_cast<int32_t>(dp[c_star] >> 32);
  if (gpus_used) *gpus_used = c_star;
  int c = c_star;
  for (int i = n_requests - 1; i >= 0; --i) {
    const Cand& o = cands[i][pick[i][c]];
    chosen[i] = o.option;
    if (steps_done) steps_done[i] = o.q;
    c -= o.width;
  }
  return DIT_OK;
}
