"""CPU oracle for the paper's round scheduler (TEST INFRASTRUCTURE, not a product path).

Plain definitions, written out:
  * `round_best` is the per-round problem of Section 5.2.2 ("select at most one option per request,
    with total GPU <= N, maximizing the number of requests that survive to the next round") solved
    by exhaustive enumeration of every combination of options; Algorithm 1's dynamic program must
    reach the same optimum (it is exact for this group knapsack).
  * `allocate_best` enumerates every split of a request's steps over one or two parallelism degrees
    and keeps the cheapest one (GPU time) that meets the budget (Section 5.2.1); `allocate_any`
    enumerates every split over ALL degrees (the unrestricted optimum, a lower bound).
Only small instances: the enumerations are exponential.
"""
from __future__ import annotations

import itertools
import math
from typing import List, Sequence, Tuple

Option = Tuple[int, int, float]          # (steps s, gpus A, step time T(A))


def option_progress(opt: Option, tau: float) -> int:
    """q = min(s, floor(tau / T(A)))  (Section 5.2.2)."""
    s, _, t = opt
    return min(s, math.floor(tau / t))


def survives(options: Sequence[Option], choice: int, t_min: float, deadline: float, tau: float, t_now: float) -> bool:
    """t_{r+1} + LB(o) <= D with LB(o) = (remaining steps after option o) * T_min."""
    remaining = sum(o[0] for o in options)
    if choice >= 0:
        remaining -= option_progress(options[choice], tau)
    return t_now + tau + remaining * t_min <= deadline


def round_best(reqs, n_gpus: int, tau: float, t_now: float):
    """reqs: list of (options, t_min, deadline).  Returns (max survivors, list of optimal plans)."""
    per_req = []
    for options, _, _ in reqs:
        ok = [-1] + [m for m, o in enumerate(options) if option_progress(o, tau) > 0 and o[1] <= n_gpus]
        per_req.append(ok)
    best, plans = -1, []
    for plan in itertools.product(*per_req):
        used = sum(reqs[i][0][m][1] for i, m in enumerate(plan) if m >= 0)
        if used > n_gpus:
            continue
        value = sum(survives(reqs[i][0], m, reqs[i][1], reqs[i][2], tau, t_now) for i, m in enumerate(plan))
        if value > best:
            best, plans = value, [plan]
        elif value == best:
            plans.append(plan)
    return best, plans


def round_best_progress(reqs, n_gpus: int, tau: float, t_now: float):
    """Among the plans with the most survivors, those that complete the most steps in the round.
    Returns (survivors, steps, plans)."""
    best, plans = round_best(reqs, n_gpus, tau, t_now)
    steps = [sum(option_progress(reqs[i][0][m], tau) for i, m in enumerate(p) if m >= 0) for p in plans]
    top = max(steps) if steps else 0
    return best, top, [p for p, s in zip(plans, steps) if s == top]


def allocate_best(gpus: Sequence[int], step_time: Sequence[float], steps: int, budget: float):
    """Cheapest split over at most two degrees: returns (gpu_time, completion_time) or None if infeasible."""
    best = None
    n = len(gpus)
    for a in range(n):
        for b in range(n):
            for na in range(steps + 1):
                nb = steps - na
                t = na * step_time[a] + nb * step_time[b]
                if t > budget:
                    continue
                cost = na * gpus[a] * step_time[a] + nb * gpus[b] * step_time[b]
                if best is None or (cost, t) < best:
                    best = (cost, t)
    return best


def allocate_any(gpus: Sequence[int], step_time: Sequence[float], steps: int, budget: float):
    """Cheapest split over any number of degrees (lower bound for `allocate_best`)."""
    best = None
    n = len(gpus)

    def rec(d, left, t, cost):
        nonlocal best
        if d == n - 1:
            t2 = t + left * step_time[d]
            c2 = cost + left * gpus[d] * step_time[d]
            if t2 <= budget and (best is None or c2 < best):
                best = c2
            return
        for k in range(left + 1):
            rec(d + 1, left - k, t + k * step_time[d], cost + k * gpus[d] * step_time[d])
    rec(0, steps, 0.0, 0.0)
    return best
