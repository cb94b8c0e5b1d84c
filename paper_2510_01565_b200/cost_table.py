"""Cost table of the paper's scheduler, filled from this library's own step.

The scheduler plans with a table T(resolution, k): the latency of one denoising step of a request
at that resolution on k GPUs, profiled offline (Section 5.2.1: step latency is deterministic per
(resolution, degree), so a profiled table predicts it; GPU cost of a step is k * T).  Here the k = 1
column is MEASURED by running the library's step on the current GPU with CUDA events; columns for
k > 1 cannot be measured on one GPU and come from a stated model of sequence parallelism (compute
divides by k, every block adds all-to-all exchanges of the request's activations), so they are
synthetic.  `plan_round` then feeds the table to the C library's allocation and round DP exactly as
the paper's control loop does at a round boundary.

Host-side logic only; the measuring function needs a CUDA device and the built library.
"""
from __future__ import annotations

import json
import math
from dataclasses import dataclass, field
from typing import Dict, List, Sequence, Tuple

import numpy as np

from . import workloads as W


@dataclass
class ParallelModel:
    """T(k) = T(1) / k + (k > 1) * n_blocks * exchanges * (latency + bytes / bandwidth), with
    bytes = tokens * hidden * 2 / k per GPU and exchange (the volume one all-to-all of a request's
    activations moves off each GPU, to first order).  Defaults: four all-to-alls per block (Q, K, V
    in, attention output back), 20 us per exchange, 450 GB/s effective per GPU."""
    exchanges_per_block: int = 4
    latency_s: float = 20e-6
    bandwidth_Bps: float = 450e9

    def overhead(self, tokens: int, hidden: int, n_blocks: int, k: int) -> float:
        if k <= 1:
            return 0.0
        per = self.latency_s + tokens * hidden * 2.0 / k / self.bandwidth_Bps
        return n_blocks * self.exchanges_per_block * per


@dataclass
class CostTable:
    hidden: int
    n_blocks: int
    n_text: int
    degrees: Tuple[int, ...] = (1, 2, 4, 8)
    t1: Dict[int, float] = field(default_factory=dict)        # resolution -> seconds per step at k = 1 (measured)
    cv: Dict[int, float] = field(default_factory=dict)        # resolution -> coefficient of variation of the measurement
    model: ParallelModel = field(default_factory=ParallelModel)

    def tokens(self, res: int) -> int:
        return (res // W.PATCH_PIXELS) ** 2 + self.n_text

    def step_time(self, res: int, k: int) -> float:
        return self.t1[res] / k + self.model.overhead(self.tokens(res), self.hidden, self.n_blocks, k)

    def gpu_time(self, res: int, k: int) -> float:
        """GPU-seconds one step costs at degree k: k * T(res, k)."""
        return k * self.step_time(res, k)

    def t_min(self, res: int) -> float:
        return min(self.step_time(res, k) for k in self.degrees)

    def to_json(self) -> str:
        rows = {str(r): {"t1_ms": 1e3 * self.t1[r], "cv": self.cv.get(r),
                         "T_ms": {str(k): 1e3 * self.step_time(r, k) for k in self.degrees},
                         "source": {str(k): "measured" if k == 1 else "model" for k in self.degrees}}
                for r in sorted(self.t1)}
        return json.dumps({"hidden": self.hidden, "n_blocks": self.n_blocks, "n_text": self.n_text, "table": rows})


def measure_k1(dims: W.ModelDims, n_blocks: int, resolutions: Sequence[int], n_text: int = 512,
               steps: int = 20, warmup: int = 3, drawn_blocks: int = 2, seed: int = 0) -> CostTable:
    """Profiles one request per resolution through `n_blocks` blocks (the drawn blocks' tensors are
    loaded cyclically: every block costs the same).  Each of `steps` steps is timed on its own with
    CUDA events; the table keeps the mean and the coefficient of variation."""
    import torch
    from . import binding as B

    table = CostTable(dims.hidden, n_blocks, n_text)
    max_tokens = max(table.tokens(r) for r in resolutions)
    ctx = B.context_for(dims, n_blocks, max_tokens, 1)
    wl0 = W.make_custom("profile", dims, min(drawn_blocks, n_blocks), [(resolutions[0], resolutions[0], n_text)], seed=seed)
    B.upload_weights(ctx, [wl0.weights[b % len(wl0.weights)] for b in range(n_blocks)])
    stream = torch.cuda.current_stream()
    for res in resolutions:
        wl = W.make_custom("profile", dims, 0, [(res, res, n_text)], seed=seed, with_weights=False)
        tok, cond = B.bits_to_cuda_bf16(wl.packed_tokens()), B.bits_to_cuda_bf16(wl.cond)
        out = torch.empty((wl.total_tokens, dims.hidden), dtype=torch.float32, device="cuda")
        for _ in range(warmup):
            ctx.dit_step_forward(tok, wl.token_lens, cond, n_blocks, out=out)
        torch.cuda.synchronize()
        events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for e0, e1 in events:
            e0.record(stream)
            ctx.dit_step_forward(tok, wl.token_lens, cond, n_blocks, out=out)
            e1.record(stream)
        torch.cuda.synchronize()
        ctx.dit_ctx_poll_status()
        ms = np.array([e0.elapsed_time(e1) for e0, e1 in events])
        table.t1[res] = float(ms.mean()) * 1e-3
        table.cv[res] = float(ms.std() / ms.mean())
    ctx.close()
    return table


@dataclass
class PendingRequest:
    resolution: int
    steps_left: int
    deadline: float        # absolute, seconds


def plan_round(queue: Sequence[PendingRequest], table: CostTable, n_gpus: int, tau: float, t_now: float):
    """One scheduling decision at a round boundary: deadline-aware allocation per request (at most two
    degrees that meet its remaining time at least GPU cost), then the round DP over the GPUs.
    Returns a list of dicts (resolution, gpus, steps this round, options) in queue order and the
    number of requests that are not definitely late after the round."""
    from . import binding as B

    degrees = [k for k in table.degrees if k <= n_gpus]
    reqs, opts_all = [], []
    for q in queue:
        times = [table.step_time(q.resolution, k) for k in degrees]
        options, _, _ = B.dit_sched_allocate(degrees, times, q.steps_left, q.deadline - t_now)
        opts_all.append(options)
        reqs.append((options, table.t_min(q.resolution), q.deadline))
    chosen, done, survivors, used = B.dit_sched_round(reqs, n_gpus, tau, t_now)
    plan = []
    for q, options, c, d in zip(queue, opts_all, chosen, done):
        plan.append({"resolution": q.resolution, "gpus": options[c][1] if c >= 0 else 0, "steps": d, "options": options})
    return plan, survivors, used


def main():
    import argparse
    ap = argparse.ArgumentParser(description="Measure the k = 1 column of the scheduler's cost table and plan one round with it")
    ap.add_argument("--blocks", type=int, default=8)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--gpus", type=int, default=8, help="GPUs the planned round assumes (the measurement uses one)")
    args = ap.parse_args()
    from . import build
    build.build_library()
    table = measure_k1(W.LARGE, args.blocks, list(W.RESOLUTIONS), steps=args.steps)
    print(table.to_json())
    # a queue like the paper's mixed workload: 50-step requests, deadlines proportional to the k = 1 run time
    rng = np.random.default_rng(0)
    queue = [PendingRequest(r, 50, 1.5 * 50 * table.t1[r]) for r in W.draw_mixed_resolutions(rng, 12)]
    tau = 5 * table.t1[1024]
    plan, survivors, used = plan_round(queue, table, args.gpus, tau, 0.0)
    print(json.dumps({"round_length_s": tau, "gpus": args.gpus, "gpus_used": used, "survivors": survivors, "plan": plan}))


if __name__ == "__main__":
    main()
