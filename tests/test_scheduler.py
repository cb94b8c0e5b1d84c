"""The paper's round scheduler (CPU library) against exhaustive enumeration and hand cases."""
import ctypes as C
import os
import re
import time

import numpy as np
import pytest

from oracle import sched_oracle as S
from paper_2510_01565_b200 import binding as B
from paper_2510_01565_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def lib():
    build.build_library()
    return B.load_library()


def test_header_symbols_exported(lib):
    header = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "dit_sched.h")).read(), flags=re.S)
    declared = set(re.findall(r"\b(dit_sched_[a-z_0-9]+)\s*\(", header))
    assert declared == set(B.SCHED_EXPORTS)
    for name in declared:
        assert hasattr(lib, name)


# ------------------------------------------------------------------ oracle pins (hand cases)
def test_oracle_hand_cases():
    # q = min(s, floor(tau / T))
    assert S.option_progress((5, 2, 0.3), 1.0) == 3 and S.option_progress((2, 2, 0.3), 1.0) == 2
    assert S.option_progress((5, 1, 1.5), 1.0) == 0
    # survival: t_next + remaining * t_min <= D.  4 steps left, t_min 0.5, round [0,1): none -> 1 + 2.0 = 3.0
    opts = [(4, 1, 0.5)]
    assert S.survives(opts, -1, 0.5, 3.0, 1.0, 0.0) and not S.survives(opts, -1, 0.5, 2.9, 1.0, 0.0)
    # running the option finishes 2 steps: 1 + 2 * 0.5 = 2.0
    assert S.survives(opts, 0, 0.5, 2.0, 1.0, 0.0) and not S.survives(opts, 0, 0.5, 1.9, 1.0, 0.0)
    # two requests that each need 2 GPUs now, 2 GPUs in total: exactly one survives
    r = ([(2, 2, 0.5)], 0.5, 1.0)          # must finish both steps in this round
    best, plans = S.round_best([r, r], 2, 1.0, 0.0)
    assert best == 1 and sorted(plans) == [(-1, 0), (0, -1)]
    best, _ = S.round_best([r, r], 4, 1.0, 0.0)
    assert best == 2
    # a request that is safe without running frees the GPUs for the urgent one
    safe = ([(2, 2, 0.5)], 0.5, 10.0)
    best, plans = S.round_best([safe, r], 2, 1.0, 0.0)
    assert best == 2 and (-1, 0) in plans
    # allocation: 10 steps, T(1)=1.0, T(2)=0.6: budget 10 -> all on 1 GPU (cost 10); budget 8 -> 5 + 5 (cost 5 + 6)
    assert S.allocate_best([1, 2], [1.0, 0.6], 10, 10.0) == (10.0, 10.0)
    cost, t = S.allocate_best([1, 2], [1.0, 0.6], 10, 8.0)
    assert cost == pytest.approx(11.0) and t == pytest.approx(8.0)
    assert S.allocate_best([1, 2], [1.0, 0.6], 10, 5.9) is None
    assert S.allocate_any([1, 2], [1.0, 0.6], 10, 8.0) == pytest.approx(11.0)


# ------------------------------------------------------------------ library vs oracle
def _random_instance(rng, n_req, n_gpus):
    reqs = []
    for _ in range(n_req):
        base = float(rng.choice([0.05, 0.12, 0.4, 1.1]))
        table = {k: base / (k ** float(rng.uniform(0.5, 0.95))) for k in (1, 2, 4, 8)}
        n_opt = int(rng.integers(0, 3))
        degs = rng.choice([1, 2, 4, 8], size=n_opt, replace=False) if n_opt else []
        options = [(int(rng.integers(0, 8)), int(k), table[int(k)]) for k in degs]
        t_min = min(table.values())
        total = sum(o[0] for o in options)
        deadline = float(rng.uniform(0.2, 1.5)) + total * t_min * float(rng.uniform(0.6, 1.6))
        reqs.append((options, t_min, deadline))
    return reqs


def test_round_dp_matches_exhaustive_search():
    rng = np.random.default_rng(0)
    for trial in range(300):
        n_gpus = int(rng.choice([1, 2, 4, 8]))
        reqs = _random_instance(rng, int(rng.integers(0, 7)), n_gpus)
        tau, t_now = float(rng.choice([0.25, 0.5, 1.0])), float(rng.uniform(0, 3))
        chosen, done, surv, used = B.dit_sched_round(reqs, n_gpus, tau, t_now)
        best, steps, plans = S.round_best_progress(reqs, n_gpus, tau, t_now)
        assert surv == best, (trial, reqs, n_gpus, tau, t_now)
        assert sum(done) == steps                          # and, among those, the most steps this round
        assert tuple(chosen) in plans                      # a valid optimal plan (several may exist)
        assert used == sum(reqs[i][0][m][1] for i, m in enumerate(chosen) if m >= 0) <= n_gpus
        for i, m in enumerate(chosen):
            assert done[i] == (S.option_progress(reqs[i][0][m], tau) if m >= 0 else 0)
            assert m == -1 or done[i] > 0


def test_round_special_cases():
    assert B.dit_sched_round([], 8, 1.0, 0.0) == ([], [], 0, 0)
    r = ([(2, 2, 0.5)], 0.5, 1.0)
    chosen, done, surv, used = B.dit_sched_round([r, r], 2, 1.0, 0.0)
    assert surv == 1 and used == 2 and sorted(chosen) == [-1, 0] and sorted(done) == [0, 2]
    # an option wider than the machine is never chosen; zero GPUs: nothing runs
    chosen, _, surv, used = B.dit_sched_round([([(1, 16, 0.1)], 0.1, 100.0)], 8, 1.0, 0.0)
    assert chosen == [-1] and surv == 1 and used == 0
    chosen, _, _, used = B.dit_sched_round([r], 0, 1.0, 0.0)
    assert chosen == [-1] and used == 0
    lib = B.load_library()
    assert lib.dit_sched_round(None, 1, 8, 1.0, 0.0, None, None, None, None) == 1
    assert lib.dit_sched_round(None, 0, 8, 0.0, 0.0, None, None, None, None) == 1      # tau must be positive


def test_allocation_matches_exhaustive_search():
    rng = np.random.default_rng(1)
    for _ in range(200):
        n = int(rng.integers(1, 5))
        gpus = [1, 2, 4, 8][:n]
        base = float(rng.uniform(0.05, 1.0))
        times = [base / (k ** float(rng.uniform(0.3, 1.0))) for k in gpus]
        steps = int(rng.integers(0, 12))
        budget = float(rng.uniform(0.2, 1.2)) * steps * base
        opts, cost, feasible = B.dit_sched_allocate(gpus, times, steps, budget)
        want = S.allocate_best(gpus, times, steps, budget)
        assert feasible == (want is not None)
        assert sum(o[0] for o in opts) == steps and len(opts) <= 2
        got_cost = sum(s * a * t for (s, a, t) in opts)
        assert cost == pytest.approx(got_cost)
        if want is not None:
            assert cost == pytest.approx(want[0], rel=1e-12)
            assert sum(s * t for (s, _, t) in opts) <= budget + 1e-12
            assert cost >= S.allocate_any(gpus, times, steps, budget) - 1e-12       # two degrees cannot beat the free optimum
        else:
            fastest = int(np.argmin(times))
            assert opts == [(steps, gpus[fastest], times[fastest])]


def test_decision_latency_is_far_below_the_papers_bound():
    """The paper reports < 10 ms per scheduling decision (Table 5); 64 requests on 8 GPUs here."""
    rng = np.random.default_rng(2)
    reqs = _random_instance(rng, 64, 8)
    t0 = time.perf_counter()
    for _ in range(20):
        B.dit_sched_round(reqs, 8, 0.5, 0.0)
    ms = (time.perf_counter() - t0) / 20 * 1e3
    assert ms < 10.0, ms
