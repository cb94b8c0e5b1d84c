"""Seeded random stacks against the oracle: block forms, variant flags, request counts and shapes are
drawn, so that combinations no hand-written case lists still meet the per-request bar (max / rms <= 1e-2
for fp16 operands; the bars of the e4m3 mode against the quantising oracle, which test_gpu_variants.py states)."""
import numpy as np
import pytest

from oracle import dit_oracle as O
from oracle import fp8_oracle as F8
from paper_2510_01565_b200 import workloads as W

import test_gpu_variants as TV

pytestmark = pytest.mark.gpu

B = TV.B        # the module-scoped binding fixture


def draw_case(rng, dims, max_requests, max_blocks):
    n = int(rng.integers(1, max_requests + 1))
    big = rng.random() < 0.4
    reqs = []
    for _ in range(n):
        if big:      # several 128-row tiles and a ragged tail
            reqs.append((16 * int(rng.integers(4, 20)), 16 * int(rng.integers(4, 20)), int(rng.integers(0, 200))))
        else:        # down to a single token row
            reqs.append((16 * int(rng.integers(1, 8)), 16 * int(rng.integers(1, 8)), int(rng.integers(0, 40))))
    fp8 = rng.random() < 0.2
    # s = sequential, p = parallel, d = two-stream (the e4m3 mode does not cover two-stream blocks)
    kinds = "".join(rng.choice(list("sp" if fp8 else "spd")) for _ in range(int(rng.integers(1, max_blocks + 1))))
    flags = int(rng.integers(0, 4)) | (4 if fp8 else 0)
    return reqs, kinds, flags, fp8, int(rng.integers(0, 10**6))


def run_case(B, dims, reqs, kinds, flags, fp8, seed):
    wl = TV.dual_stack_workload(dims, kinds, reqs, seed=seed, qk_norm=bool(flags & 1))
    ctx, out, slots, tok, cond = TV.run_stack(B, wl, flags)
    pos = [O.patch_positions(q.height, q.width, q.n_text_tokens) for q in wl.requests] if flags & 2 else None
    if fp8:      # every linear product of every block in e4m3
        ref = F8.step_forward_fp8(W.bf16_to_f64(wl.packed_tokens()), wl.token_lens, W.bf16_to_f64(wl.cond), TV.f64_blocks(wl),
                                  wl.dims.n_heads, wl.dims.ln_eps, positions=pos)
    else:
        ref = O.step_forward(W.bf16_to_f64(wl.packed_tokens()), wl.token_lens, W.bf16_to_f64(wl.cond), TV.f64_blocks(wl),
                             wl.dims.n_heads, wl.dims.ln_eps, positions=pos,
                             n_imgs=[q.n_image_tokens for q in wl.requests])
    mx, rms = TV.worst_errors(wl, out, ref)
    ctx.close()
    return mx, rms


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_stacks_small_model(B, seed):
    rng = np.random.default_rng(seed)
    for _ in range(6):
        reqs, kinds, flags, fp8, s = draw_case(rng, W.SMALL, 8, 3)
        mx, rms = run_case(B, W.SMALL, reqs, kinds, flags, fp8, s)
        what = f"requests {reqs} blocks {kinds} flags {flags} seed {s}: max {mx:.2e} rms {rms:.2e}"
        if fp8:
            assert rms <= TV.FP8_RMS_QUANTISED and mx <= TV.FP8_MAX_QUANTISED, what
        else:
            assert mx <= 1e-2, what


def test_random_stacks_large_model(B):
    rng = np.random.default_rng(21)
    for _ in range(3):
        reqs, kinds, flags, fp8, s = draw_case(rng, W.LARGE, 3, 2)
        mx, rms = run_case(B, W.LARGE, reqs, kinds, flags, fp8, s)
        what = f"requests {reqs} blocks {kinds} flags {flags} seed {s}: max {mx:.2e} rms {rms:.2e}"
        if fp8:
            assert rms <= TV.FP8_RMS_QUANTISED and mx <= TV.FP8_MAX_QUANTISED, what
        else:
            assert mx <= 1e-2, what
