"""The scheduler's cost table and the round-planning glue (host logic; the k = 1 column is measured on a GPU
in the gpu-marked test)."""
import math

import numpy as np
import pytest

from oracle import sched_oracle as S
from paper_2510_01565_b200 import build, cost_table as CT, workloads as W


@pytest.fixture(scope="module", autouse=True)
def lib():
    build.build_library()


def fake_table():
    t = CT.CostTable(hidden=3072, n_blocks=8, n_text=512)
    t.t1 = {256: 0.004, 512: 0.008, 1024: 0.030, 2048: 0.200}
    return t


def test_table_arithmetic():
    t = fake_table()
    assert t.tokens(1024) == 4096 + 512 and t.tokens(256) == 256 + 512
    # k = 1 is the measurement itself; k > 1 divides the compute and adds the exchange model
    for r in t.t1:
        assert t.step_time(r, 1) == t.t1[r]
        for k in (2, 4, 8):
            over = 8 * 4 * (20e-6 + t.tokens(r) * 3072 * 2.0 / k / 450e9)
            assert t.step_time(r, k) == pytest.approx(t.t1[r] / k + over, rel=1e-12)
            assert t.gpu_time(r, k) == pytest.approx(k * t.step_time(r, k), rel=1e-12)
            assert t.gpu_time(r, k) > t.gpu_time(r, 1)          # parallelism never saves GPU time in this model
    # large requests scale, small ones do not: the paper's observation that motivates per-request degrees
    eff = lambda r, k: t.step_time(r, 1) / (k * t.step_time(r, k))
    assert eff(2048, 8) > 0.9 and eff(256, 8) < 0.5 and eff(256, 8) < eff(512, 8) < eff(1024, 8) < eff(2048, 8)
    assert t.t_min(2048) == t.step_time(2048, 8)


def test_plan_round_matches_the_oracle():
    t = fake_table()
    rng = np.random.default_rng(0)
    for trial in range(20):
        n = int(rng.integers(1, 6))
        queue = [CT.PendingRequest(int(rng.choice([256, 512, 1024, 2048])), int(rng.integers(1, 12)), 0.0) for _ in range(n)]
        for q in queue:
            q.deadline = float(rng.uniform(0.6, 2.5)) * q.steps_left * t.t1[q.resolution]
        n_gpus, tau = 8, 5 * t.t1[1024]
        plan, survivors, used = CT.plan_round(queue, t, n_gpus, tau, 0.0)
        # the same decision from the oracles: allocation per request, then exhaustive search of the round
        reqs = []
        for q, p in zip(queue, plan):
            times = [t.step_time(q.resolution, k) for k in t.degrees]
            best = S.allocate_best(list(t.degrees), times, q.steps_left, q.deadline)
            cost = sum(s * a * tt for (s, a, tt) in p["options"])
            if best is not None:
                assert cost == pytest.approx(best[0], rel=1e-9)
            assert sum(s for (s, _, _) in p["options"]) == q.steps_left
            reqs.append((p["options"], t.t_min(q.resolution), q.deadline))
        want, _ = S.round_best(reqs, n_gpus, tau, 0.0)
        assert survivors == want
        assert used == sum(p["gpus"] for p in plan) <= n_gpus
        for q, p in zip(queue, plan):
            if p["gpus"]:
                opt = [o for o in p["options"] if o[1] == p["gpus"]][0]
                assert p["steps"] == min(opt[0], math.floor(tau / opt[2])) > 0
            else:
                assert p["steps"] == 0


@pytest.mark.gpu
def test_measured_column_on_the_gpu():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    t = CT.measure_k1(W.LARGE, 2, [256, 512, 1024], steps=10)
    assert t.t1[256] < t.t1[512] < t.t1[1024]
    assert all(cv < 0.15 for cv in t.cv.values()), t.cv           # step latency is predictable (Section 5.2.1)
    # quadrupling the image tokens costs at least twice and (attention grows quadratically) more than 4x only at scale
    assert 2.0 < t.t1[1024] / t.t1[512] < 6.0
    queue = [CT.PendingRequest(r, 20, 2.0 * 20 * t.t1[r]) for r in (256, 512, 1024, 1024)]
    plan, survivors, used = CT.plan_round(queue, t, 4, 5 * t.t1[1024], 0.0)
    assert survivors == 4 and 0 < used <= 4
    assert '"measured"' in t.to_json()
