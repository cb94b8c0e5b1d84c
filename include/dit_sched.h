/*
 * Round scheduler of the paper (CPU only, no GPU code): deadline-aware GPU allocation and the
 * per-round dynamic program that picks, for every pending request, at most one of its allocation
 * options so that as many requests as possible are not "definitely late" at the next round start
 * (Section 5.2 "Round-Based Scheduling", Algorithm 1 "DP Round Scheduler").
 *
 * All pointers are HOST memory owned by the caller; nothing is allocated beyond the call's own
 * stack/heap temporaries and nothing is retained.  Times are in one unit of the caller's choice.
 */
#ifndef DIT_SCHED_H_
#define DIT_SCHED_H_

#include <stdint.h>

#include "dit.h"

#ifdef __cplusplus
extern "C" {
#endif

/* One allocation option (s_i^m, A_i^m) of a request with its profiled step time T_i(A_i^m). */
typedef struct {
  int32_t steps;    /* s_i^m >= 0: remaining steps planned at this degree */
  int32_t gpus;     /* A_i^m >= 1: GPUs the option occupies in a round */
  double step_time; /* T_i(A_i^m) > 0 */
} dit_sched_option;

typedef struct {
  const dit_sched_option *options; /* [n_options] */
  int32_t n_options;
  double t_min;    /* T_i^min = min_k T_i(k): fastest possible step time of this request */
  double deadline; /* D_i, absolute */
} dit_sched_request;

/* Deadline-aware GPU allocation (Section 5.2.1): for one request with `steps` remaining steps and
 * profiled step times step_time[d] on gpus[d] GPUs (d = 0..n_degrees-1, e.g. 1, 2, 4, 8), find the
 * split of the steps over AT MOST TWO degrees (the form the paper's allocations take) that minimises
 * the GPU time sum_m s^m * A^m * T(A^m) subject to sum_m s^m * T(A^m) <= time_budget (queueing delay
 * is not modelled).  Writes 1 or 2 options to out (zero-step options are dropped) and the GPU time.
 * If even the fastest degree misses the budget, *feasible = 0 and the result is all steps at the
 * fastest degree.  Ties: fewer GPU-seconds, then shorter completion time, then lower degrees.
 * DIT_ERR_INVALID_ARG on NULL pointers, n_degrees < 1, steps < 0, non-positive times or GPU counts. */
dit_status dit_sched_allocate(const int32_t *gpus, const double *step_time, int32_t n_degrees, int32_t steps,
                              double time_budget, dit_sched_option *out /*[2]*/, int32_t *n_out, double *gpu_time,
                              int32_t *feasible);

/* Algorithm 1.  For round [t_now, t_now + tau) on n_gpus GPUs: option m of request i can complete
 * q = min(s_i^m, floor(tau / T_i(A_i^m))) steps; options with q = 0 or A_i^m > n_gpus are dropped;
 * a request survives option o (or "none") iff t_now + tau + (remaining steps after o) * T_i^min <= D_i;
 * a group-knapsack DP over capacities 0..n_gpus maximises the number of survivors with at most one
 * option per request.  Among plans with that many survivors the one that completes the most steps in
 * the round is taken (the paper reaches a work-conserving plan through a separate scale-up pass over
 * idle GPUs; here the DP's value is the pair (survivors, steps) compared in that order, so GPUs are
 * not left idle while a request could use them).  Remaining ties: the plan found by scanning requests
 * in order, capacities upward and options in order (none first), keeping the first maximum.
 * Outputs (each may be NULL except chosen): chosen[i] = option index or -1 for "none", steps_done[i] =
 * q of the choice (0 for none), the number of survivors and the GPUs used.  O(R * N * options) time. */
dit_status dit_sched_round(const dit_sched_request *reqs, int32_t n_requests, int32_t n_gpus, double tau, double t_now,
                           int32_t *chosen, int32_t *steps_done, int32_t *n_survivors, int32_t *gpus_used);

#ifdef __cplusplus
}
#endif
#endif /* DIT_SCHED_H_ */
