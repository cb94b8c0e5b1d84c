"""The N > 1 path of the benchmark on CPU: two gloo ranks, max-over-ranks timing, whole-job rate."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp

from paper_2510_01565_b200 import replicas
from paper_2510_01565_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist = replicas.init_process_group("gloo")
    # every rank draws the same seeded batch: replicas process identical work (weak scaling)
    wl = W.make_workload("cfg1_small_256", with_weights=False)
    dist.barrier()
    ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    slowest = replicas.max_over_ranks(ms, dist)
    rate = replicas.whole_job_rate(wl.image_tokens, world, slowest)
    dist.barrier()
    q.put((rank, slowest, rate, wl.total_tokens))
    dist.destroy_process_group()


def test_two_replicas_report_slowest_rank_and_aggregate_rate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, rate, tokens in got:
        assert slowest == 15.0
        assert rate == pytest.approx(2 * 256 / 0.015)
        assert tokens == 256


def test_single_process_passthrough():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rate(100, 4, 20.0) == pytest.approx(20000.0)
