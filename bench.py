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

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, transcribed from
# the committed ncu summaries (profiles/); None until a capture exists for that workload.
# Captured on cfg3_1024x2 (profiles/gemm_tcgen05_dram_traffic_cfg3_1024x2.md): 530 MB per launch averaged over the
# four GEMMs of a block; traffic is proportional to T, so other workloads of the 3072-wide model scale by T / 9216.
NCU_TRAFFIC_BYTES_PER_TOKEN_3072 = 530.0e6 / 9216


def ncu_traffic(wl):
    if wl.dims.hidden != 3072:
        return None
    return NCU_TRAFFIC_BYTES_PER_TOKEN_3072 * wl.total_tokens


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
                                          "--format=csv,noheader,nounits", "-lms", "100"],
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
    """The oracle, as it stands, timed on the host cores (rank 0 only)."""
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
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * wl.n_blocks * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "n_blocks": wl.n_blocks, "sample": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


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
    build.build_library()
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
    slots = nb * (2 if args.form == "dual" else 1)     # a two-stream block takes two weight slots
    ctx = B.context_for(wl.dims, slots, wl.total_tokens, len(wl.requests), flags=args.variants)
    assert B.upload_weights(ctx, wl.weights) == slots
    lens = wl.token_lens
    tok_bits, cond_bits = wl.packed_tokens(), wl.cond
    tok, cond = B.bits_to_cuda_bf16(tok_bits), B.bits_to_cuda_bf16(cond_bits)
    out = torch.empty((wl.total_tokens, wl.dims.hidden), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()
    needs_geometry = bool(args.variants & 2) or args.form == "dual"
    if args.variants or needs_geometry:
        # the rotary term and two-stream blocks need each token's place in its request: the step is given the requests
        step = lambda: ctx.dit_step_forward_requests(tok, wl.requests, cond, slots, out=out)
    else:
        step = lambda: ctx.dit_step_forward(tok, lens, cond, slots, out=out)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms: float) -> float:
        return replicas.max_over_ranks(ms, dist, "cuda")

    # ---------------------------------------------------------------- device-resident throughput
    for _ in range(args.warmup):
        step()
    barrier()
    ctx.dit_ctx_poll_status()
    sampler = ClockSampler(local_rank)
    sampler.start()
    ctx.dit_ctx_set_timing(True)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    clocks = sampler.stop()
    kernels = ctx.dit_ctx_read_timing()
    ctx.dit_ctx_set_timing(False)
    ctx.dit_ctx_poll_status()
    launches = ctx.dit_last_launch_count() * args.steps
    ms_step = ms_total / args.steps
    img_tokens = wl.image_tokens * world
    value = replicas.whole_job_rate(wl.image_tokens, world, ms_step)
    flops = wl.flops_per_step()
    tflops = flops / (ms_step * 1e-3) / 1e12

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
        barrier()
        e0.record(stream)
        for _ in range(args.steps):
            g.replay()
        e1.record(stream)
        barrier()
        graph_ms = max_over_ranks(e0.elapsed_time(e1)) / args.steps
    except Exception as exc:   # graph capture is a convenience figure, never the headline
        sys.stderr.write(f"cuda graph timing skipped: {exc}\n")

    # ---------------------------------------------------------------- end to end with host buffers
    h_tok = torch.from_numpy(tok_bits.view(np.int16)).pin_memory()
    h_cond = torch.from_numpy(cond_bits.view(np.int16)).pin_memory()
    h_out = torch.empty((wl.total_tokens, wl.dims.hidden), dtype=torch.float32).pin_memory()
    e2e_steps = max(1, min(args.steps, 5))

    def e2e_step():
        if needs_geometry:        # the host-buffer entry point carries no geometry: copy, run, copy back by hand
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
    e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps
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

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---------------------------------------------------------------- per-kernel figures and the roofline
    peaks = measured_peaks()
    H, F, T = wl.dims.hidden, wl.dims.mlp_hidden, wl.total_tokens
    per_launch_flops = {"gemm_qkv": 2.0 * T * H * 3 * H, "gemm_proj": 2.0 * T * H * H, "gemm_fc1": 2.0 * T * H * F,
                        "gemm_fc2": 2.0 * T * H * (F + (H if args.form == "parallel" else 0)),   # parallel form: one K = H + F output GEMM
                        "attention": 4.0 * H * sum(l * l for l in lens)}
    per_launch_bytes = {"ln_modulate": T * H * (4 + 2), "modulation": slots * wl.dims.cond_dim * 6 * H * 2}
    kern = {}
    for name, rec in kernels.items():
        if not rec["launches"]:
            continue
        avg_ms = rec["ms"] / rec["launches"]
        k = {"launches": rec["launches"], "avg_ms": avg_ms, "share": rec["ms"] / (ms_step * args.steps)}
        if name in per_launch_flops:
            k["tflops"] = per_launch_flops[name] / (avg_ms * 1e-3) / 1e12
            k["frac_of_bf16_peak"] = k["tflops"] / peaks["bf16_tflops"]
        else:
            k["gbs"] = per_launch_bytes[name] / (avg_ms * 1e-3) / 1e9
            k["frac_of_hbm_peak"] = k["gbs"] / peaks["hbm_gbs"]
        kern[name] = k
    gemm_names = [n for n in ("gemm_qkv", "gemm_proj", "gemm_fc1", "gemm_fc2") if n in kern]
    gemm_ms = sum(kernels[n]["ms"] for n in gemm_names)
    gemm_launches = sum(kernels[n]["launches"] for n in gemm_names)
    gemm_flops = sum(per_launch_flops[n] * kernels[n]["launches"] for n in gemm_names)
    achieved = gemm_flops / (gemm_ms * 1e-3) / 1e12
    roofline = {"bound": "tensor", "kernel": "gemm_tcgen05_kernel (QKV, projection, FC1, FC2 launches)",
                "achieved": achieved, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_tflops_sustained"], "peak_kind": f"bf16 sustained, of {peaks['source']}",
                "frac_of_burst_peak": achieved / peaks["bf16_tflops"],
                "avg_launch_ms": gemm_ms / gemm_launches, "launches": gemm_launches,
                "traffic": ncu_traffic(wl),
                "algorithmic_bytes": (T * H * 2 * 2 + 3 * H * H * 2 + T * 3 * H * 2 + H * H * 2 + T * H * 8 + T * H * 2 + H * F * 2
                                      + T * F * 2 * 2 + F * H * 2 + T * H * 8) / 4.0}

    # the largest single kernel by time is attention: its own figure beside the GEMMs' (same peak; at d = 128
    # its exponentials need as many special-function cycles as its MMAs need tensor cycles)
    roofline_attention = None
    if "attention" in kern:
        a = kern["attention"]
        roofline_attention = {"bound": "tensor", "kernel": "attention_tcgen05_kernel", "achieved": a["tflops"],
                              "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                              "frac": a["tflops"] / peaks["bf16_tflops_sustained"], "avg_launch_ms": a["avg_ms"],
                              "launches": a["launches"], "share_of_step": a["share"],
                              "traffic": None}

    # ---------------------------------------------------------------- the oracle on the host cores
    run, n_img, desc = oracle_sample(wl)
    reps, t0 = 0, time.perf_counter()
    while reps < 8 and (reps == 0 or time.perf_counter() - t0 < 10.0):
        run()
        reps += 1
    cpu_s = (time.perf_counter() - t0) / reps
    cpu = {"value": n_img / cpu_s, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc,
           "seconds_per_sample": cpu_s, "repeats": reps}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16+e4m3 (reduced precision, not the headline)" if args.variants & 4 else "f16",
            "data": "synthetic",
            "config": {"workload": wl.name, "block_form": args.form, "block_variants": {"qk_rmsnorm": bool(args.variants & 1), "rope_2d": bool(args.variants & 2), "fp8_qkv_fc1": bool(args.variants & 4)}, "n_blocks": nb, "weights_reused_cyclically": bool(args.depth), "requests": [f"{r.height}x{r.width}+{r.n_text_tokens}" for r in wl.requests],
                       "total_tokens": T, "image_tokens": wl.image_tokens, "hidden": H, "heads": wl.dims.n_heads,
                       "head_dim": wl.dims.head_dim, "mlp_hidden": F, "parallelism": f"replicas x{world}",
                       "l2": "weights and activations of a step exceed L2 (126 MB); no flush"},
            "tflops": tflops, "frac_of_bf16_peak": tflops / peaks["bf16_tflops"],
            "frac_of_bf16_sustained": tflops / peaks["bf16_tflops_sustained"], "peaks": peaks,
            "roofline": roofline, "roofline_attention": roofline_attention, "kernels": kern, "cpu_baseline": cpu,
            "e2e": {"value": img_tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
            "cuda_graph_replay": None if graph_ms is None else {"ms_per_step": graph_ms, "value": replicas.whole_job_rate(wl.image_tokens, world, graph_ms), "unit": UNIT},
            "full_step": {"what": "latent in, latent out: conditioning + patch embedding + the block stack + final layer + Euler update",
                          "ms_per_step": full_ms, "value": replicas.whole_job_rate(wl.image_tokens, world, full_ms), "unit": UNIT,
                          "steps": full_steps, "launches_per_step": full_launches, "shell_ms": shell_ms,
                          "shell_share": sum(shell_ms.values()) / full_ms},
            "gpu_launches": launches, "clocks": clocks}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(W.CONFIGS))
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--depth", type=int, default=0, help="run this many blocks instead of the configuration's (weights reused cyclically)")
    ap.add_argument("--variants", type=int, default=0, choices=list(range(8)),
                    help="context flag bits: 1 = RMS-norm of queries and keys, 2 = 2-D rotary term, 4 = e4m3 operands for the "
                         "QKV and up-projection GEMMs (reduced precision: never the headline configuration)")
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
