"""GPU parity of the shell around the block stack (latent -> tokens, timestep -> cond, final layer,
Euler update, and the whole denoising step) against the fp64 CPU oracle, through the C ABI.

Bars: values that the library rounds to bf16 (cond, tokens) may differ from the oracle's rounding
by one bf16 step where the fp32 and fp64 pre-images fall on different sides of a rounding
boundary; velocities and latent updates use the step's bar, max|gpu - oracle| / rms(oracle) <= 1e-2
per request (measured values are far below it).
"""
import numpy as np
import pytest

from oracle import dit_oracle as O
from oracle import step_oracle as S
from paper_2510_01565_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = 1e-2
BF16_STEP = 2.0 ** -7          # spacing of bf16 relative to the power of two below |v|


@pytest.fixture(scope="module")
def B():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device; the library has no CPU path")
    from paper_2510_01565_b200 import binding, build
    build.build_library()
    binding.load_library()
    return binding


def f64w(w):
    return {k: W.bf16_to_f64(v) for k, v in w.items()}


class ShellRun:
    def __init__(self, B, si: W.StepInputs, n_blocks, flags=0):
        import torch
        self.torch, self.B, self.si, self.nb = torch, B, si, n_blocks
        total = sum(si.token_lens)
        self.ctx = B.context_for(si.dims, max(n_blocks, 1), total, max(len(si.requests), 1), flags=flags)
        if n_blocks:
            B.upload_weights(self.ctx, si.weights[:n_blocks])
        B.upload_shell_weights(self.ctx, si.shell)
        self.latents = torch.from_numpy(np.concatenate([z.reshape(-1) for z in si.latents])).cuda()
        txt = np.concatenate(si.texts, axis=0)
        self.text = B.bits_to_cuda_bf16(txt) if txt.shape[0] else None
        self.pooled = torch.from_numpy(si.pooled).cuda()
        self.lat_cu = np.concatenate([[0], np.cumsum([z.size for z in si.latents])])
        self.tok_cu = np.concatenate([[0], np.cumsum(si.token_lens)])

    def latent_of(self, flat, r):
        return flat[int(self.lat_cu[r]):int(self.lat_cu[r + 1])].cpu().numpy().astype(np.float64).reshape(self.si.latents[r].shape)

    def sync(self):
        self.torch.cuda.synchronize()
        self.ctx.dit_ctx_poll_status()

    def close(self):
        self.ctx.close()


def assert_bf16_close(got, want, what):
    """got, want: fp64 arrays of bf16-representable values; at most one bf16 step apart."""
    step = BF16_STEP * np.maximum(np.abs(want), 2.0 ** -20)
    bad = np.abs(got - want) > 1.001 * step
    assert not bad.any(), f"{what}: {int(bad.sum())} values differ by more than one bf16 step"
    frac = float((got != want).mean())
    assert frac < 0.02, f"{what}: {frac:.3%} of the values differ from the oracle's rounding"


MIXED_SMALL = [(64, 96, 5), (32, 32, 0), (128, 64, 17), (16, 16, 1), (96, 160, 0)]


def test_timestep_cond_matches_oracle(B):
    si = W.make_step_inputs(W.SMALL, 0, MIXED_SMALL, seed=11)
    run = ShellRun(B, si, 0)
    shell = f64w(si.shell)
    for pooled in (run.pooled, None):
        cond = run.ctx.dit_timestep_cond(si.requests, pooled)
        run.sync()
        got = cond.float().cpu().numpy().astype(np.float64)
        for r, q in enumerate(si.requests):
            pre = S.timestep_cond(q.timestep, si.pooled[r].astype(np.float64) if pooled is not None else None, shell)
            assert O.error_metric(got[r], pre) <= 2.0 ** -6        # fp32 result rounded to bf16
            assert_bf16_close(got[r], S.round_to_bf16(pre), f"cond of request {r}")
    run.close()


def test_embed_latents_matches_oracle(B):
    si = W.make_step_inputs(W.SMALL, 0, MIXED_SMALL, seed=12)
    run = ShellRun(B, si, 0)
    shell = f64w(si.shell)
    tok = run.ctx.dit_embed_latents(run.latents, run.text, si.requests)
    run.sync()
    got = tok.float().cpu().numpy().astype(np.float64)
    assert got.shape == (sum(si.token_lens), W.SMALL.hidden)
    for r, q in enumerate(si.requests):
        rows = got[int(run.tok_cu[r]):int(run.tok_cu[r + 1])]
        want_img = S.round_to_bf16(S.embed_latent(si.latents[r].astype(np.float64), shell, W.SMALL.hidden))
        assert_bf16_close(rows[:q.n_image_tokens], want_img, f"image tokens of request {r}")
        assert np.array_equal(rows[q.n_image_tokens:], W.bf16_to_f64(si.texts[r])), f"text rows of request {r}"
    run.close()


def test_embed_of_a_request_does_not_depend_on_its_neighbours(B):
    si = W.make_step_inputs(W.SMALL, 0, MIXED_SMALL, seed=13)
    run = ShellRun(B, si, 0)
    tok = run.ctx.dit_embed_latents(run.latents, run.text, si.requests)
    run.sync()
    r = 2
    q = si.requests[r]
    z = run.latents[int(run.lat_cu[r]):int(run.lat_cu[r + 1])].contiguous()
    txt = B.bits_to_cuda_bf16(si.texts[r])
    alone = run.ctx.dit_embed_latents(z, txt, [q])
    run.sync()
    assert run.torch.equal(alone, tok[int(run.tok_cu[r]):int(run.tok_cu[r + 1])])
    run.close()


def test_final_layer_and_sampler_update_match_oracle(B):
    si = W.make_step_inputs(W.SMALL, 0, MIXED_SMALL, seed=14)
    run = ShellRun(B, si, 0)
    torch = run.torch
    shell = f64w(si.shell)
    rng = np.random.default_rng(5)
    total = sum(si.token_lens)
    x = (rng.standard_normal((total, W.SMALL.hidden)) * 2.0 + 0.5).astype(np.float32)
    cond_bits = W.f32_to_bf16_bits(rng.standard_normal((len(si.requests), W.SMALL.cond_dim)).astype(np.float32))
    vel = run.ctx.dit_final_layer(torch.from_numpy(x).cuda(), si.requests, B.bits_to_cuda_bf16(cond_bits))
    run.sync()
    want_v = []
    for r, q in enumerate(si.requests):
        a = int(run.tok_cu[r])
        v_tok = S.final_layer(x[a:a + q.n_image_tokens].astype(np.float64), W.bf16_to_f64(cond_bits[r]), shell, W.SMALL.ln_eps)
        want = S.unpatchify(v_tok, q.height // 8, q.width // 8)
        want_v.append(want)
        err = O.error_metric(run.latent_of(vel, r), want)
        assert err <= TOL, f"velocity of request {r}: {err:.3e}"
    # sampler: z + dsigma * v with the GPU's own v is a single fused multiply-add per element
    before = run.latents.clone()
    run.ctx.dit_sampler_update(run.latents, vel, si.requests, si.dsigmas)
    run.sync()
    for r in range(len(si.requests)):
        z0, v = run.latent_of(before, r), run.latent_of(vel, r)
        want = S.euler_update(z0, v, float(si.dsigmas[r]))
        assert np.abs(run.latent_of(run.latents, r) - want).max() <= 2.0 ** -22 * max(1.0, np.abs(want).max())
    run.close()


def _oracle_step(si, n_blocks, latents=None):
    return S.denoise_step([z.astype(np.float64) for z in (latents or si.latents)],
                          [W.bf16_to_f64(t) for t in si.texts], [q.timestep for q in si.requests],
                          [float(d) for d in si.dsigmas], [p.astype(np.float64) for p in si.pooled],
                          f64w(si.shell), [f64w(w) for w in si.weights[:n_blocks]], si.dims.n_heads, si.dims.ln_eps)


def check_step(run, si, n_blocks, tol=TOL):
    torch = run.torch
    before = run.latents.clone()
    vel = torch.empty_like(run.latents)
    run.ctx.dit_denoise_step(run.latents, run.text, si.requests, si.dsigmas, run.pooled, n_blocks, velocity=vel)
    run.sync()
    assert run.ctx.dit_last_launch_count() == (1 + 7 * n_blocks) + 8
    new, vels, _ = _oracle_step(si, n_blocks)
    for r in range(len(si.requests)):
        err = O.error_metric(run.latent_of(vel, r), vels[r])
        assert err <= tol, f"velocity of request {r}: {err:.3e}"
        dz_got = run.latent_of(run.latents, r) - run.latent_of(before, r)
        dz_want = new[r] - si.latents[r].astype(np.float64)
        err = O.error_metric(dz_got, dz_want)
        assert err <= tol, f"latent update of request {r}: {err:.3e}"
    return before, vel


def test_denoise_step_small_mixed_batch(B):
    si = W.make_step_inputs(W.SMALL, 2, MIXED_SMALL, seed=15)
    run = ShellRun(B, si, 2)
    before, vel = check_step(run, si, 2)
    # the one-call step equals the five calls made one after another, bit for bit
    ctx, torch = run.ctx, run.torch
    cond = ctx.dit_timestep_cond(si.requests, run.pooled)
    tok = ctx.dit_embed_latents(before, run.text, si.requests)
    x = ctx.dit_step_forward(tok, si.token_lens, cond, 2)
    v2 = ctx.dit_final_layer(x, si.requests, cond)
    z2 = before.clone()
    ctx.dit_sampler_update(z2, v2, si.requests, si.dsigmas)
    run.sync()
    assert torch.equal(v2, vel)
    assert torch.equal(z2, run.latents)
    run.close()


def test_denoise_step_large_dims_with_text(B):
    # the serving model's width (3072, 24 heads of 128) on a 256^2 and a 512x256 request with text
    si = W.make_step_inputs(W.LARGE, 2, [(256, 256, 64), (512, 256, 0)], seed=16)
    run = ShellRun(B, si, 2)
    check_step(run, si, 2)
    run.close()


def test_denoise_step_with_bf16_operands(B):
    # the whole step in the bf16-operand mode: the final layer's LayerNorm output and output projection take the
    # mode's formats too; bar of the mode (6e-2), and the velocity differs from the fp16-operand step's
    si = W.make_step_inputs(W.SMALL, 2, MIXED_SMALL, seed=19)
    run16 = ShellRun(B, si, 2)
    _, vel16 = check_step(run16, si, 2)
    run16.close()
    run = ShellRun(B, si, 2, flags=B.DIT_FLAG_BF16_OPERANDS)
    _, vel = check_step(run, si, 2, tol=6e-2)
    assert not run.torch.equal(vel, vel16)
    run.close()


def test_three_steps_of_a_schedule_follow_the_oracle(B):
    # the latent is carried from step to step, as a served request's is; errors must not build up
    reqs = [(64, 64, 3), (32, 96, 0)]
    si = W.make_step_inputs(W.SMALL, 2, reqs, seed=17)
    run = ShellRun(B, si, 2)
    z_ref = [z.astype(np.float64) for z in si.latents]
    sigmas = [1.0, 0.7, 0.4, 0.15]
    start = [z.copy() for z in z_ref]
    for s, s_next in zip(sigmas[:-1], sigmas[1:]):
        qs = [W.Request(q.height, q.width, q.n_text_tokens, 1000.0 * s, 0) for q in si.requests]
        ds = np.full(len(qs), s_next - s, dtype=np.float32)
        run.ctx.dit_denoise_step(run.latents, run.text, qs, ds, run.pooled, 2)
        z_ref, _, _ = S.denoise_step(z_ref, [W.bf16_to_f64(t) for t in si.texts], [q.timestep for q in qs],
                                     [float(d) for d in ds], [p.astype(np.float64) for p in si.pooled],
                                     f64w(si.shell), [f64w(w) for w in si.weights[:2]], si.dims.n_heads, si.dims.ln_eps)
    run.sync()
    for r in range(len(reqs)):
        moved_got = run.latent_of(run.latents, r) - start[r]
        moved_want = z_ref[r] - start[r]
        err = O.error_metric(moved_got, moved_want)
        assert err <= TOL, f"request {r} after three steps: {err:.3e}"
    run.close()


def test_shell_argument_errors(B):
    si = W.make_step_inputs(W.SMALL, 1, [(32, 32, 0)], seed=18)
    torch = __import__("torch")
    ctx = B.context_for(W.SMALL, 1, 64, 2)
    z = torch.zeros(64 * 4, device="cuda")
    with pytest.raises(B.DitError) as e:                      # shell weights not loaded yet
        ctx.dit_embed_latents(z, None, si.requests)
    assert e.value.status == 4
    B.upload_shell_weights(ctx, si.shell)
    with pytest.raises(B.DitError) as e:                      # block weights not loaded
        ctx.dit_denoise_step(z, None, si.requests, [-0.1], None, 1)
    assert e.value.status == 4
    with pytest.raises(B.DitError) as e:                      # a request with text but no text buffer
        ctx.dit_embed_latents(z, None, [(32, 32, 3, 0.0)])
    assert e.value.status == 1
    with pytest.raises(B.DitError) as e:                      # resolution not a multiple of 16
        ctx.dit_timestep_cond([(40, 32, 0, 1.0)])
    assert e.value.status == 2
    with pytest.raises(B.DitError) as e:                      # more tokens than the context holds
        ctx.dit_timestep_cond([(256, 256, 0, 1.0)])
    assert e.value.status == 3
    assert ctx.dit_timestep_cond([]).shape == (0, W.SMALL.cond_dim)   # empty batch: nothing to do
    torch.cuda.synchronize()
    ctx.dit_ctx_poll_status()
    ctx.close()


def test_round_with_uneven_step_counts(B):
    # one scheduling round on a worker: each request runs its own number of steps, the packed batch
    # shrinks as requests use up their quota (the second request runs no step at all)
    import torch
    reqs = [(64, 96, 5), (32, 32, 0), (96, 32, 2), (32, 64, 7)]
    si = W.make_step_inputs(W.SMALL, 2, reqs, seed=19)
    run = ShellRun(B, si, 2)
    steps = [3, 0, 1, 2]
    sig = np.zeros((4, 4), dtype=np.float32)
    for r, start in enumerate([1.0, 0.5, 0.62, 0.3]):
        sig[r] = np.float32(start) - np.float32(0.07) * np.arange(4, dtype=np.float32) * np.float32(1 + 0.1 * r)
    before = run.latents.clone()
    run.ctx.dit_denoise_round(run.latents, run.text, si.requests, steps, sig, run.pooled, 2)
    run.sync()
    assert run.ctx.dit_last_launch_count() == 3 * ((1 + 7 * 2) + 8)
    shell, blocks = f64w(si.shell), [f64w(w) for w in si.weights[:2]]
    for r in range(4):
        z = si.latents[r].astype(np.float64)
        for k in range(steps[r]):
            t = float(np.float32(1000.0) * sig[r, k])
            ds = float(sig[r, k + 1] - sig[r, k])
            (z,), _, _ = S.denoise_step([z], [W.bf16_to_f64(si.texts[r])], [t], [ds], [si.pooled[r].astype(np.float64)],
                                        shell, blocks, si.dims.n_heads, si.dims.ln_eps)
        got = run.latent_of(run.latents, r)
        if steps[r] == 0:
            assert np.array_equal(got, si.latents[r].astype(np.float64))       # untouched
        else:
            err = O.error_metric(got - si.latents[r].astype(np.float64), z - si.latents[r].astype(np.float64))
            assert err <= TOL, f"request {r} after {steps[r]} steps: {err:.3e}"
    # the same round as separate steps on the shrinking request lists, bit for bit
    z2 = before.clone()
    for k in range(3):
        act = [r for r in range(4) if steps[r] > k]
        qs = [W.Request(si.requests[r].height, si.requests[r].width, si.requests[r].n_text_tokens,
                        float(np.float32(1000.0) * sig[r, k]), 0) for r in act]
        lat = torch.cat([z2[int(run.lat_cu[r]):int(run.lat_cu[r + 1])] for r in act])
        txt = [B.bits_to_cuda_bf16(si.texts[r]) for r in act if si.texts[r].shape[0]]
        txt = torch.cat(txt) if txt else None
        ds = np.array([sig[r, k + 1] - sig[r, k] for r in act], dtype=np.float32)
        run.ctx.dit_denoise_step(lat, txt, qs, ds, run.pooled[act].contiguous(), 2)
        p = 0
        for r in act:
            m = int(run.lat_cu[r + 1] - run.lat_cu[r])
            z2[int(run.lat_cu[r]):int(run.lat_cu[r + 1])] = lat[p:p + m]
            p += m
    run.sync()
    assert torch.equal(z2, run.latents)
    run.close()
