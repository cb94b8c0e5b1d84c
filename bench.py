#!/usr/bin/env python
"""Benchmark of the single-GPU DiT denoising step (image tokens/s, fraction of the bf16 tensor roofline).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5_mixed8] [--impl reference]

A "step" is one pass of the whole hot path (modulation, LayerNorm+modulate, QKV GEMM, varlen
attention, projection, MLP, for every block of the stack) over one packed batch of synthetic
requests.  Rank 0 prints ONE JSON line.  With N > 1 (launched by torch.distributed.run) every rank
runs an independent replica of the same batch: the path has no exchange step, so there is no
data-path collective; timing is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2510_01565_b200 import workloads as W  # noqa: E402

METRIC = "dit_step_image_tokens_per_s"
UNIT = "image tokens/s"
DEFAULT_WORKLOAD = "cfg5_mixed8"

# dram__bytes_read.sum + dram__bytes_write.sum per launch, from ncu captures of the 2 x 1024^2 step (T = 9216
# packed rows of the 3072-wide model; the summaries under profiles/ give the commands).  GEMM: average over the
# four GEMMs of a block.  Both kernels read every activation row once and the weights (GEMM) or a request's
# keys and values (attention) once per band of rows that fits L2, so traffic grows with T and other workloads
# of the same model are scaled by T / 9216; `traffic_scaled_from` in the JSON line says so.
NCU_CAPTURE_TOKENS = 9216
NCU_GEMM_TRAFFIC_BYTES = 509.0e6
NCU_ATTENTION_TRAFFIC_BYTES = 205.0e6


def ncu_traffic(wl, bytes_at_capture):
    if wl.dims.hidden != 3072:
        return None, None
    scale = wl.total_tokens / NCU_CAPTURE_TOKENS
    origin = ("ncu capture of cfg3_1024x2" if wl.total_tokens == NCU_CAPTURE_TOKENS
              else f"ncu capture of cfg3_1024x2, scaled by T / {NCU_CAPTURE_TOKENS} = {scale:.3f}")
    return bytes_at_capture * scale, origin


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16_tflops": p["bf16_tflops"], "bf16_tflops_sustained": p["bf16_tflops_sustained"],
                "hbm_gbs": p["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(wl: W.Workload):
    """A bounded piece of the workload for the CPU oracle: its smallest request through ONE block.

    Returns (run, image_tokens_per_step_equivalent, description): every block of the stack costs the
    same, so one block's time times the stack depth is the request's step time; the returned token
    count is already divided by the depth, i.e. tokens / seconds(run) is image tokens per second of
    a full-depth step.
    """
    from oracle import dit_oracle as O
    r = int(np.argmin(wl.token_lens))
    x = W.bf16_to_f64(wl.tokens[r])
    c = W.bf16_to_f64(wl.cond[r])
    w0 = {k: W.bf16_to_f64(v) for k, v in wl.weights[0].items() if k != "txt"}
    if "txt" in wl.weights[0]:
        w0["txt"] = {k: W.bf16_to_f64(v) for k, v in wl.weights[0]["txt"].items()}
    req = wl.requests[r]

    def run():
        return O.any_block_forward(x, c, w0, wl.dims.n_heads, wl.dims.ln_eps, n_img=req.n_image_tokens)
    desc = (f"request {r} of {wl.name} alone ({req.height}x{req.width}: {req.n_image_tokens} image + "
            f"{req.n_text_tokens} text tokens) through 1 of {wl.n_blocks} blocks, time scaled by {wl.n_blocks}; fp64 NumPy")
    return run, req.n_image_tokens / wl.n_blocks, desc


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    """The oracle, as it stands, timed on the host cores (rank 0 only).

    One "step" of this arm is a bounded sample (the workload's smallest request through one block);
    `value` is the sample's image tokens divided by the measured sample time and by the stack depth,
    and `ms_per_step` is that sample time multiplied by the depth: an extrapolation, flagged as such,
    with the measured seconds beside it.
    """
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = W.make_workload(args.workload, seed=args.seed, n_blocks_drawn=1)
    run, n_img, desc = oracle_sample(wl)
    for _ in range(args.warmup):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = (time.perf_counter() - t0) / args.steps
    value = n_img / dt
    cores = blas_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * wl.n_blocks * 1e3,
            "ms_per_step_is": f"extrapolated: measured seconds per sample x {wl.n_blocks} blocks, one request only",
            "measured_seconds_per_sample": dt, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "n_blocks": wl.n_blocks, "sample": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                             "seconds_per_sample": dt},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


MIN_REGION_SECONDS = 2.0     # a timed region shorter than this gives the 50 ms clock sampler too few samples


class DeviceBench:
    """One workload resident on the device: timed regions of whole steps with per-kernel events and a clock record."""

    def __init__(self, B, torch, replicas, dist, local_rank, world, wl, args, form="sequential", variants=0):
        self.B, self.torch, self.replicas, self.dist, self.local_rank, self.world = B, torch, replicas, dist, local_rank, world
        self.wl, self.form, self.variants = wl, form, variants
        nb = wl.n_blocks
        self.slots = nb * (2 if form == "dual" else 1)     # a two-stream block takes two weight slots
        self.ctx = B.context_for(wl.dims, self.slots, wl.total_tokens, len(wl.requests), flags=variants)
        assert B.upload_weights(self.ctx, wl.weights) == self.slots
        self.lens = wl.token_lens
        self.tok_bits, self.cond_bits = wl.packed_tokens(), wl.cond
        self.tok, self.cond = B.bits_to_cuda_bf16(self.tok_bits), B.bits_to_cuda_bf16(self.cond_bits)
        self.out = torch.empty((wl.total_tokens, wl.dims.hidden), dtype=torch.float32, device="cuda")
        self.stream = torch.cuda.current_stream()
        self.needs_geometry = bool(variants & 2) or form == "dual"
        ctx, tok, cond, out, slots = self.ctx, self.tok, self.cond, self.out, self.slots
        if variants & 7 or self.needs_geometry:
            # the rotary term and two-stream blocks need each token's place in its request: the step is given the requests
            self.step = lambda: ctx.dit_step_forward_requests(tok, wl.requests, cond, slots, out=out)
        else:
            self.step = lambda: ctx.dit_step_forward(tok, self.lens, cond, slots, out=out)
        self.e0, self.e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def max_over_ranks(self, ms: float) -> float:
        return self.replicas.max_over_ranks(ms, self.dist, "cuda")

    def region(self, fn, n_steps, per_kernel=False):
        """Times exactly n_steps calls of fn between two barriers; returns (ms per step, clock record, kernel times)."""
        sampler = ClockSampler(self.local_rank)
        sampler.start()
        if per_kernel:
            self.ctx.dit_ctx_set_timing(True)
            self.ctx.dit_debug_clock_probe(True)         # the SM clock attention and GEMM CTAs really run at inside the step
        self.barrier()
        self.e0.record(self.stream)
        for _ in range(n_steps):
            fn()
        self.e1.record(self.stream)
        self.barrier()
        ms = self.max_over_ranks(self.e0.elapsed_time(self.e1)) / n_steps
        clocks = sampler.stop()
        kernels = None
        if per_kernel:
            kernels = self.ctx.dit_ctx_read_timing()
            self.ctx.dit_ctx_set_timing(False)
            self.clock_probe = self.ctx.dit_debug_clock_probe(False)
        self.ctx.dit_ctx_poll_status()
        return ms, clocks, kernels

    def kernel_table(self, kernels, ms_step, n_steps, peaks):
        wl = self.wl
        H, F, T = wl.dims.hidden, wl.dims.mlp_hidden, wl.total_tokens
        flops = {"gemm_qkv": 2.0 * T * H * 3 * H, "gemm_proj": 2.0 * T * H * H, "gemm_fc1": 2.0 * T * H * F,
                 "gemm_fc2": 2.0 * T * H * (F + (H if self.form == "parallel" else 0)),   # parallel form: one K = H + F output GEMM
                 "attention": 4.0 * H * sum(l * l for l in self.lens)}
        nbytes = {"ln_modulate": T * H * (4 + 2), "modulation": self.slots * wl.dims.cond_dim * 6 * H * 2,
                  # e4m3 mode: fp16 in, codes out, two launches per block (attention output, GELU output; one for a parallel block)
                  "quantize": T * (H + F) * 3 / (1 if self.form == "parallel" else 2)}
        kern = {}
        for name, rec in kernels.items():
            if not rec["launches"]:
                continue
            avg_ms = rec["ms"] / rec["launches"]
            k = {"launches": rec["launches"], "avg_ms": avg_ms, "share": rec["ms"] / (ms_step * n_steps)}
            if name in flops:
                k["tflops"] = flops[name] / (avg_ms * 1e-3) / 1e12
                k["frac_of_bf16_peak"] = k["tflops"] / peaks["bf16_tflops"]
            else:
                k["gbs"] = nbytes[name] / (avg_ms * 1e-3) / 1e9
                k["frac_of_hbm_peak"] = k["gbs"] / peaks["hbm_gbs"]
            kern[name] = k
        return kern, flops

    def rooflines(self, kern, kernels, flops, peaks):
        wl = self.wl
        H, F, T = wl.dims.hidden, wl.dims.mlp_hidden, wl.total_tokens
        gemm_names = [n for n in ("gemm_qkv", "gemm_proj", "gemm_fc1", "gemm_fc2") if n in kern]
        gemm_ms = sum(kernels[n]["ms"] for n in gemm_names)
        gemm_launches = sum(kernels[n]["launches"] for n in gemm_names)
        gemm_flops = sum(flops[n] * kernels[n]["launches"] for n in gemm_names)
        achieved = gemm_flops / (gemm_ms * 1e-3) / 1e12
        traffic, origin = ncu_traffic(wl, NCU_GEMM_TRAFFIC_BYTES)
        roofline = {"bound": "tensor", "kernel": "gemm_tcgen05_kernel (QKV, projection, FC1, FC2 launches)",
                    "achieved": achieved, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                    "frac": achieved / peaks["bf16_tflops_sustained"],
                    "peak_kind": f"bf16 sustained (the kernel is timed inside a long step), of {peaks['source']}",
                    "frac_of_burst_peak": achieved / peaks["bf16_tflops"],
                    "avg_launch_ms": gemm_ms / gemm_launches, "launches": gemm_launches,
                    "traffic": traffic, "traffic_scaled_from": origin,
                    "algorithmic_bytes": (T * H * 2 * 2 + 3 * H * H * 2 + T * 3 * H * 2 + H * H * 2 + T * H * 8 + T * H * 2 + H * F * 2
                                          + T * F * 2 * 2 + F * H * 2 + T * H * 8) / 4.0}
        # the largest single kernel by time is attention: its own figure beside the GEMMs' (same peaks; at d = 128
        # its exponentials need as many special-function cycles as its MMAs need tensor cycles)
        roofline_attention = None
        if "attention" in kern:
            a = kern["attention"]
            atraffic, aorigin = ncu_traffic(wl, NCU_ATTENTION_TRAFFIC_BYTES)
            roofline_attention = {"bound": "tensor", "kernel": "attention_tcgen05_kernel", "achieved": a["tflops"],
                                  "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                                  "frac": a["tflops"] / peaks["bf16_tflops_sustained"],
                                  "frac_of_burst_peak": a["tflops"] / peaks["bf16_tflops"], "avg_launch_ms": a["avg_ms"],
                                  "launches": a["launches"], "share_of_step": a["share"],
                                  "traffic": atraffic, "traffic_scaled_from": aorigin,
                                  "algorithmic_bytes": T * 4 * H * 2}
        return roofline, roofline_attention

    def close(self):
        self.ctx.close()


def step_summary(bench, ms_step, n_steps, clocks, kernels, peaks):
    """The figures of one timed region of whole steps: throughput, TFLOP/s, whole-step and per-kernel fractions."""
    wl = bench.wl
    tflops = wl.flops_per_step() / (ms_step * 1e-3) / 1e12
    kern, flops = bench.kernel_table(kernels, ms_step, n_steps, peaks)
    roofline, roofline_attention = bench.rooflines(kern, kernels, flops, peaks)
    # attention against the chip's peak AT THE CLOCK ITS CTAs RAN AT (the part is power-capped and clocks kernels
    # differently; nvidia-smi's samples cannot be attributed to a kernel): SMs x 8192 dense fp16 FLOP per cycle x MHz
    mhz, cyc, gemm_mhz = getattr(bench, "clock_probe", (0, 0, 0))
    sms = bench.torch.cuda.get_device_properties(bench.torch.cuda.current_device()).multi_processor_count
    how = "clock64 against %globaltimer over one CTA's life (dit_debug_clock_probe)"
    if roofline_attention is not None and mhz > 0:
        peak_at_clock = sms * 8192 * mhz * 1e6 / 1e12
        roofline_attention["in_kernel"] = {"sm_mhz": mhz, "cycles_per_key_block": cyc, "peak_at_that_clock_tflops": peak_at_clock,
                                           "frac_of_peak_at_that_clock": roofline_attention["achieved"] / peak_at_clock, "how": how}
    if gemm_mhz > 0:
        peak_at_clock = sms * 8192 * gemm_mhz * 1e6 / 1e12
        roofline["in_kernel"] = {"sm_mhz": gemm_mhz, "peak_at_that_clock_tflops": peak_at_clock,
                                 "frac_of_peak_at_that_clock": roofline["achieved"] / peak_at_clock, "how": how}
    return {"workload": wl.name, "steps": n_steps, "ms_per_step": ms_step,
            "value": bench.replicas.whole_job_rate(wl.image_tokens, bench.world, ms_step), "unit": UNIT,
            "tflops": tflops,
            # whole step (GEMMs + attention + the HBM-bound kernels) against both measured bf16 peaks
            "roofline_step": {"bound": "tensor", "achieved": tflops, "unit": "TFLOP/s", "peak": peaks["bf16_tflops"],
                              "frac": tflops / peaks["bf16_tflops"], "peak_kind": f"bf16 burst, of {peaks['source']}",
                              "frac_of_sustained_peak": tflops / peaks["bf16_tflops_sustained"]},
            "roofline": roofline, "roofline_attention": roofline_attention, "kernels": kern, "clocks": clocks,
            "timed_region_s": ms_step * n_steps * 1e-3}


def run_gpu(args):
    import torch
    from paper_2510_01565_b200 import binding as B
    from paper_2510_01565_b200 import build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    from paper_2510_01565_b200 import replicas
    dist = None
    if world > 1:
        torch.cuda.set_device(local_rank)
        dist = replicas.init_process_group("nccl", torch.device("cuda", local_rank))
    else:
        torch.cuda.set_device(0)
    # one rank compiles (if the library is stale), the others wait for it instead of racing on the same file
    if rank == 0:
        build.build_library()
    if dist is not None:
        dist.barrier()
    B.load_library()

    wl = W.make_workload(args.workload, seed=args.seed)
    nb = wl.n_blocks
    if args.depth:
        # a deeper stack than the configuration draws (e.g. 57 blocks, the depth class of the models the
        # paper serves): the drawn blocks' weights are loaded cyclically, which costs the same per block
        nb = args.depth
        wl.weights = [wl.weights[b % len(wl.weights)] for b in range(nb)]
        wl.n_blocks = nb
    if args.form == "parallel":
        par_rng = np.random.default_rng(args.seed + 3000)
        drawn = [W.draw_parallel_block_weights(par_rng, wl.dims) for _ in range(min(nb, 4))]
        wl.weights = [drawn[b % len(drawn)] for b in range(nb)]
    if args.form == "dual":
        txt_rng = np.random.default_rng(args.seed + 4000)
        drawn = [W.draw_block_weights(txt_rng, wl.dims) for _ in range(min(nb, 2))]
        wl.weights = [dict(w, txt=drawn[b % len(drawn)]) for b, w in enumerate(wl.weights)]
    if args.variants & 1:
        qk_rng = np.random.default_rng(args.seed + 2000)
        qk = W.draw_qk_norm(qk_rng, wl.dims)
        wl.weights = [dict(w, **qk, **({"txt": dict(w["txt"], **qk)} if "txt" in w else {})) for w in wl.weights]
    bench = DeviceBench(B, torch, replicas, dist, local_rank, world, wl, args, args.form, args.variants)
    ctx, step, stream, slots, lens = bench.ctx, bench.step, bench.stream, bench.slots, bench.lens
    tok, cond, out = bench.tok, bench.cond, bench.out
    barrier, max_over_ranks = bench.barrier, bench.max_over_ranks
    e0, e1 = bench.e0, bench.e1
    peaks = measured_peaks()

    # ---------------------------------------------------------------- device-resident throughput: exactly --steps steps
    for _ in range(args.warmup):
        step()
    barrier()
    ctx.dit_ctx_poll_status()
    ms_step, clocks, kernels = bench.region(step, args.steps, per_kernel=True)
    head = step_summary(bench, ms_step, args.steps, clocks, kernels, peaks)
    launches = ctx.dit_last_launch_count() * args.steps
    img_tokens = wl.image_tokens * world
    value = head["value"]
    # a region under two seconds leaves the clock sampler with too few samples: the same steps again, as many as
    # fill two seconds, reported beside the headline region with their own clock record
    extended = None
    if ms_step * args.steps < MIN_REGION_SECONDS * 1e3:
        n_ext = int(math.ceil(MIN_REGION_SECONDS * 1e3 / ms_step))
        ms_e, clocks_e, kernels_e = bench.region(step, n_ext, per_kernel=True)
        extended = step_summary(bench, ms_e, n_ext, clocks_e, kernels_e, peaks)

    # ---------------------------------------------------------------- the same step replayed from a CUDA graph
    # (the step neither allocates nor synchronises, so a caller can capture it; this removes the launch
    # overhead that dominates the small-resolution steps)
    graph_ms = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            step()
        stream.wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step()
        for _ in range(args.warmup):
            g.replay()
        n_graph = max(args.steps, int(math.ceil(0.5e3 / ms_step)))
        graph_ms, _, _ = bench.region(g.replay, n_graph)
    except Exception as exc:   # graph capture is a convenience figure, never the headline
        sys.stderr.write(f"cuda graph timing skipped: {exc}\n")

    # ---------------------------------------------------------------- end to end with host buffers
    h_tok = torch.from_numpy(bench.tok_bits.view(np.int16)).pin_memory()
    h_cond = torch.from_numpy(bench.cond_bits.view(np.int16)).pin_memory()
    h_out = torch.empty((wl.total_tokens, wl.dims.hidden), dtype=torch.float32).pin_memory()
    e2e_steps = max(1, min(args.steps, 5))

    def e2e_step():
        if bench.needs_geometry:        # the host-buffer entry point carries no geometry: copy, run, copy back by hand
            tok.copy_(h_tok.view(torch.bfloat16), non_blocking=True)
            cond.copy_(h_cond.view(torch.bfloat16), non_blocking=True)
            step()
            h_out.copy_(out, non_blocking=True)
            stream.synchronize()
        else:
            ctx.dit_step_forward_host(h_tok, lens, h_cond, slots, h_out)

    e2e_step()
    barrier()
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_serial_ms = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps
    # the same with two steps in flight (dit_step_forward_host_async / dit_host_wait): step k + 1's tokens go in under
    # step k, step k's output goes out under step k + 1; every step still copies its inputs in and its output out
    e2e_ms, e2e_pipelined = e2e_serial_ms, False
    if not bench.needs_geometry:
        h_out2 = [h_out, torch.empty_like(h_out).pin_memory()]
        n_pipe = max(e2e_steps, 8)

        def e2e_pipeline():
            ctx.dit_step_forward_host_async(h_tok, lens, h_cond, slots, h_out2[0])
            for k in range(1, n_pipe):
                ctx.dit_step_forward_host_async(h_tok, lens, h_cond, slots, h_out2[k & 1])
                ctx.dit_host_wait(1)
            ctx.dit_host_wait(0)

        e2e_pipeline()
        barrier()
        e0.record(stream)
        e2e_pipeline()
        e1.record(stream)          # the host has waited for the last output: the stream is idle, the stamp is taken now
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / n_pipe
        e2e_pipelined = True
        e2e_steps = n_pipe
        del h_out2
    h2d = h_tok.numel() * 2 + h_cond.numel() * 2
    d2h = h_out.numel() * 4

    # ---------------------------------------------------------------- the full step: latent in, latent out
    # (conditioning, patch embedding, the same block stack, final layer, Euler update; the shell's
    # tensors are drawn from their own generator so that the step-only inputs above are unchanged)
    shell_rng = np.random.default_rng(args.seed + 1000)
    B.upload_shell_weights(ctx, W.draw_shell_weights(shell_rng, wl.dims))
    n_lat = 64 * wl.image_tokens
    latents = torch.randn(n_lat, device="cuda", generator=torch.Generator(device="cuda").manual_seed(args.seed))
    n_txt = sum(r.n_text_tokens for r in wl.requests)
    text = torch.randn((n_txt, wl.dims.hidden), device="cuda").to(torch.bfloat16) if n_txt else None
    pooled = torch.randn((len(wl.requests), wl.dims.cond_dim), device="cuda")
    dsig = np.full(len(wl.requests), -0.02, dtype=np.float32)

    def timed_ms(fn, reps):
        fn()
        barrier()
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1)) / reps

    full_steps = max(1, min(args.steps, 5))
    full_ms = timed_ms(lambda: ctx.dit_denoise_step(latents, text, wl.requests, dsig, pooled, slots), full_steps)
    full_launches = ctx.dit_last_launch_count()
    cond_dev = ctx.dit_timestep_cond(wl.requests, pooled)
    shell_ms = {"timestep_cond": timed_ms(lambda: ctx.dit_timestep_cond(wl.requests, pooled, cond_out=cond_dev), 5),
                "embed_latents": timed_ms(lambda: ctx.dit_embed_latents(latents, text, wl.requests, packed_tokens=tok), 5)}
    vel = torch.empty_like(latents)
    shell_ms["final_layer"] = timed_ms(lambda: ctx.dit_final_layer(out, wl.requests, cond_dev, velocity=vel), 5)
    shell_ms["sampler_update"] = timed_ms(lambda: ctx.dit_sampler_update(latents, vel, wl.requests, dsig), 5)
    ctx.dit_ctx_poll_status()
    bench.close()
    del bench, ctx, tok, cond, out, h_tok, h_out, latents, vel, text
    torch.cuda.empty_cache()

    # ---------------------------------------------------------------- the other half of the metric
    # The metric names two workloads, the 1024^2 step and the mixed-resolution packed step.  The headline above is
    # the one --workload selects (default: the mixed step); the other one is measured here in the same process, in
    # a region of at least two seconds, and reported under "secondary".
    secondary = None
    other = {"cfg5_mixed8": "cfg3_1024x2", "cfg3_1024x2": "cfg5_mixed8"}.get(args.workload)
    if other and not args.no_secondary and not args.depth and args.form == "sequential" and not args.variants:
        wl2 = W.make_workload(other, seed=args.seed)
        b2 = DeviceBench(B, torch, replicas, dist, local_rank, world, wl2, args)
        for _ in range(args.warmup):
            b2.step()
        est, _, _ = b2.region(b2.step, 3)
        n2 = max(args.steps, int(math.ceil(MIN_REGION_SECONDS * 1e3 / est)))
        ms2, clocks2, kernels2 = b2.region(b2.step, n2, per_kernel=True)
        if rank == 0:
            secondary = step_summary(b2, ms2, n2, clocks2, kernels2, peaks)
            secondary["config"] = {"workload": wl2.name, "n_blocks": wl2.n_blocks, "total_tokens": wl2.total_tokens,
                                   "image_tokens": wl2.image_tokens,
                                   "requests": [f"{r.height}x{r.width}+{r.n_text_tokens}" for r in wl2.requests]}
        b2.close()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    H, F, T = wl.dims.hidden, wl.dims.mlp_hidden, wl.total_tokens
    tflops = head["tflops"]

    # ---------------------------------------------------------------- the oracle on the host cores
    run, n_img, desc = oracle_sample(wl)
    reps, t0 = 0, time.perf_counter()
    while reps < 8 and (reps == 0 or time.perf_counter() - t0 < 10.0):
        run()
        reps += 1
    cpu_s = (time.perf_counter() - t0) / reps
    cpu = {"value": n_img / cpu_s, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc,
           "seconds_per_sample": cpu_s, "repeats": reps}

    dtype = "f16"
    if args.variants & 4:
        dtype = "f16+e4m3 (reduced precision, not the headline)"
    if args.variants & 8:
        dtype = "bf16 operands (coarser than the headline's fp16 operands)"
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": dtype, "data": "synthetic",
            "config": {"workload": wl.name, "block_form": args.form,
                       "block_variants": {"qk_rmsnorm": bool(args.variants & 1), "rope_2d": bool(args.variants & 2),
                                          "fp8_all_gemms": bool(args.variants & 4), "bf16_operands": bool(args.variants & 8)},
                       "n_blocks": nb, "weights_reused_cyclically": bool(args.depth),
                       "requests": [f"{r.height}x{r.width}+{r.n_text_tokens}" for r in wl.requests],
                       "total_tokens": T, "image_tokens": wl.image_tokens, "hidden": H, "heads": wl.dims.n_heads,
                       "head_dim": wl.dims.head_dim, "mlp_hidden": F, "parallelism": f"replicas x{world}",
                       "l2": "weights and activations of a step exceed L2 (126 MB); no flush"},
            "tflops": tflops, "frac_of_bf16_peak": tflops / peaks["bf16_tflops"],
            "frac_of_bf16_sustained": tflops / peaks["bf16_tflops_sustained"], "peaks": peaks,
            "roofline": head["roofline"], "roofline_attention": head["roofline_attention"], "roofline_step": head["roofline_step"],
            "kernels": head["kernels"], "cpu_baseline": cpu,
            "e2e": {"value": img_tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "how": ("dit_step_forward_host_async with two steps in flight: every step copies its tokens and cond in from "
                            "pinned host memory and its output back, the copies of neighbouring steps overlap the compute")
                           if e2e_pipelined else "dit_step_forward_host, one step at a time",
                    "one_step_at_a_time": {"ms_per_step": e2e_serial_ms, "value": img_tokens / (e2e_serial_ms * 1e-3)}},
            "cuda_graph_replay": None if graph_ms is None else {"ms_per_step": graph_ms, "value": replicas.whole_job_rate(wl.image_tokens, world, graph_ms), "unit": UNIT},
            "full_step": {"what": "latent in, latent out: conditioning + patch embedding + the block stack + final layer + Euler update",
                          "ms_per_step": full_ms, "value": replicas.whole_job_rate(wl.image_tokens, world, full_ms), "unit": UNIT,
                          "steps": full_steps, "launches_per_step": full_launches, "shell_ms": shell_ms,
                          "shell_share": sum(shell_ms.values()) / full_ms},
            "gpu_launches": launches, "clocks": clocks, "timed_region_s": head["timed_region_s"],
            "extended": extended, "secondary": secondary}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=25)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(W.CONFIGS))
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--depth", type=int, default=0, help="run this many blocks instead of the configuration's (weights reused cyclically)")
    ap.add_argument("--variants", type=int, default=0, choices=list(range(9)),
                    help="context flag bits: 1 = RMS-norm of queries and keys, 2 = 2-D rotary term, 4 = e4m3 operands for the "
                         "GEMMs (reduced precision: never the headline configuration), 8 = bf16 operands (alone)")
    ap.add_argument("--no-secondary", action="store_true",
                    help="skip the second workload of the metric (the 1024^2 step beside the mixed step, or vice versa)")
    ap.add_argument("--form", default="sequential", choices=["sequential", "parallel", "dual"],
                    help="block form: the adaLN-Zero block of the headline, the parallel attention+MLP form, or the "
                         "two-stream form with separate image/text tensors (same FLOPs each; not the headline)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
