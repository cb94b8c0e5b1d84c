"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle.

Bar (per request): max|gpu - oracle| / rms(oracle) <= 1e-2 on the step output.
Integer results and packed-vs-alone GPU outputs must be bit-identical.

Every run of the helper below first fills the activation regions of the workspace with NaN bytes
(`dit_debug_poison`), so a kernel that reads a row nobody wrote shows up as NaN in the output, and
checks the guard areas between the regions afterwards (the stand-in for a memory checker).

The long requests (1024^2 and 2048^2 through 4 and 8 blocks) are compared at full depth with oracle
rows stored in tests/golden/deep_rows.npz (written by tests/golden/make_deep_rows.py from the oracle
alone); for those the maximum runs over the stored rows and the rms is the oracle's over the whole
request (also stored), and over the stored rows.
"""
import os

import numpy as np
import pytest

from oracle import dit_oracle as O
from paper_2510_01565_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = 1e-2   # max|gpu - oracle| / rms(oracle), per request

DEEP_ROWS = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "deep_rows.npz")


def check_deep_rows(run, out, cfg, r):
    """Full-depth comparison of request r with the stored oracle rows of configuration `cfg`."""
    with np.load(DEEP_ROWS) as z:
        rows, ref = z[f"{cfg}/r{r}/rows"], z[f"{cfg}/r{r}/out"].astype(np.float64)
        rms_full, rms_rows = float(z[f"{cfg}/r{r}/rms_full"]), float(z[f"{cfg}/r{r}/rms_rows"])
        assert int(z[f"{cfg}/r{r}/n_tokens"]) == run.wl.token_lens[r] and int(z[f"{cfg}/r{r}/n_blocks"]) == run.nb
    got = run.rows(out, r)[run.torch.from_numpy(rows.astype(np.int64)).cuda()].cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    dmax = float(np.abs(got - ref).max())
    err_full, err_rows = dmax / rms_full, dmax / rms_rows
    print(f"{cfg} request {r}: max|d|/rms over {len(rows)} stored rows = {err_full:.3e} (request rms), {err_rows:.3e} (rows' rms)")
    assert err_full <= TOL and err_rows <= TOL, f"{cfg} request {r}: {err_full:.3e} / {err_rows:.3e}"
    return err_full


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


def oracle_requests(wl, which, n_blocks=None, taps=None):
    """Oracle outputs for the requests in `which`, converting one block's weights at a time."""
    nb = wl.n_blocks if n_blocks is None else n_blocks
    xs = {r: W.bf16_to_f64(wl.tokens[r]) for r in which}
    for b in range(nb):
        w = f64w(wl.weights[b])
        for r in which:
            tp = taps[r] if (taps is not None and b == nb - 1) else None
            xs[r] = O.block_forward(xs[r], W.bf16_to_f64(wl.cond[r]), w, wl.dims.n_heads, wl.dims.ln_eps, taps=tp)
    return xs


class DeviceRun:
    def __init__(self, B, wl, n_blocks=None, max_requests=None):
        import torch
        self.torch, self.B, self.wl = torch, B, wl
        self.nb = wl.n_blocks if n_blocks is None else n_blocks
        self.ctx = B.context_for(wl.dims, self.nb, wl.total_tokens, max_requests or max(len(wl.requests), 1))
        B.upload_weights(self.ctx, wl.weights[:self.nb])
        self.tok = B.bits_to_cuda_bf16(wl.packed_tokens())
        self.cond = B.bits_to_cuda_bf16(wl.cond)
        self.cu = np.concatenate([[0], np.cumsum(wl.token_lens)])

    def _step(self, tok, lens, cond, n_blocks):
        self.ctx.dit_debug_poison()                       # unwritten reads become NaN in the output
        out = self.ctx.dit_step_forward(tok, lens, cond, n_blocks or self.nb)
        self.torch.cuda.synchronize()
        self.ctx.dit_ctx_poll_status()
        assert self.ctx.dit_debug_check_guards() == 0, "a kernel wrote outside its region of the workspace"
        return out

    def packed(self, n_blocks=None):
        return self._step(self.tok, self.wl.token_lens, self.cond, n_blocks)

    def alone(self, r, n_blocks=None):
        a, b = int(self.cu[r]), int(self.cu[r + 1])
        return self._step(self.tok[a:b].contiguous(), [b - a], self.cond[r:r + 1].contiguous(), n_blocks)

    def rows(self, out, r):
        return out[int(self.cu[r]):int(self.cu[r + 1])]

    def close(self):
        self.ctx.close()


def check_request(run, out, r, ref):
    got = run.rows(out, r).cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    err = O.error_metric(got, ref)
    assert err <= TOL, f"request {r}: max|d|/rms = {err:.3e}"
    return err


def check_packed_equals_alone(run, out, requests=None):
    for r in (range(len(run.wl.requests)) if requests is None else requests):
        assert run.torch.equal(run.rows(out, r), run.alone(r)), f"request {r}: packed and alone outputs differ"


# ----------------------------------------------------------------------------- the five configurations
def test_cfg1_small_block_full_parity_and_taps(B):
    wl = W.make_workload("cfg1_small_256")
    run = DeviceRun(B, wl)
    out = run.packed()
    taps = {0: {}}
    ref = oracle_requests(wl, [0], taps=taps)
    check_request(run, out, 0, ref[0])
    # per-kernel intermediates (fp16 inside the library): localises a failure
    for name, key in [("qkv", "qkv"), ("attn", "a"), ("u", "u"), ("h", "h2")]:
        got = run.ctx.dit_debug_tap(name).cpu().numpy().astype(np.float64)
        assert O.error_metric(got, taps[0][key]) <= TOL, name
    mod = run.ctx.dit_debug_tap("mod").cpu().numpy().astype(np.float64)[0]
    w0 = f64w(wl.weights[0])
    want = np.concatenate(O.adaln_modulation(W.bf16_to_f64(wl.cond[0]), w0["w_ada"], w0["b_ada"]))
    assert O.error_metric(mod, want) <= 1e-5
    assert run.torch.equal(out, run.packed())          # same launch twice: bit-identical
    assert run.ctx.dit_last_launch_count() == 1 + 7 * wl.n_blocks
    run.close()


def test_cfg2_512_four_blocks(B):
    import torch
    wl = W.make_workload("cfg2_512")
    run = DeviceRun(B, wl)
    out = run.packed()
    check_request(run, out, 0, oracle_requests(wl, [0])[0])
    # the host-buffer entry point moves tokens in and the output out in row slices that overlap the
    # first and the last kernels (1536 rows = 3 slices here): same bits as the device-buffer call
    h_tok = torch.from_numpy(wl.packed_tokens().view(np.int16)).pin_memory()
    h_cond = torch.from_numpy(wl.cond.view(np.int16)).pin_memory()
    h_out = torch.full(out.shape, float("nan"), dtype=torch.float32).pin_memory()
    for _ in range(2):
        run.ctx.dit_step_forward_host(h_tok, wl.token_lens, h_cond, wl.n_blocks, h_out)
        assert torch.equal(h_out, out.cpu())
        h_out.fill_(float("nan"))
    run.ctx.dit_ctx_poll_status()
    run.close()


def test_cfg3_1024_two_requests_packed(B):
    wl = W.make_workload("cfg3_1024x2")
    run = DeviceRun(B, wl)
    out = run.packed()
    check_packed_equals_alone(run, out)
    # both requests through all 4 blocks against the stored oracle rows
    check_deep_rows(run, out, "cfg3_1024x2", 0)
    check_deep_rows(run, out, "cfg3_1024x2", 1)
    run.close()


def test_cfg4_2048_long_sequence(B):
    wl = W.make_workload("cfg4_2048")
    run = DeviceRun(B, wl)
    # one block at full length against oracle rows the CPU can produce one by one
    out1 = run.packed(n_blocks=1)
    L = wl.token_lens[0]
    rng = np.random.default_rng(0)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 129, 16383, 16384, L - 129, L - 128, L - 1],
                                     rng.integers(0, L, size=38)]))
    ref = O.block_forward(W.bf16_to_f64(wl.tokens[0]), W.bf16_to_f64(wl.cond[0]), f64w(wl.weights[0]),
                          wl.dims.n_heads, wl.dims.ln_eps, rows=rows)
    got = out1.cpu().numpy().astype(np.float64)[rows]
    assert O.error_metric(got, ref) <= TOL
    # the full 4-block step: finite, against the stored oracle rows, reproducible bit for bit
    out = run.packed()
    assert bool(run.torch.isfinite(out).all())
    check_deep_rows(run, out, "cfg4_2048", 0)
    assert run.torch.equal(out, run.packed())
    run.close()


def test_cfg5_mixed_resolution_eight_requests(B):
    wl = W.make_workload("cfg5_mixed8")
    assert [r.height for r in wl.requests] == [1024, 512, 256, 256, 1024, 2048, 1024, 1024]
    run = DeviceRun(B, wl)
    out = run.packed()
    assert bool(run.torch.isfinite(out).all())
    check_packed_equals_alone(run, out)
    # full 8-block oracle on the requests the CPU finishes quickly: 256^2 (x2) and 512^2
    ref = oracle_requests(wl, [1, 2, 3])
    for r in (1, 2, 3):
        check_request(run, out, r, ref[r])
    # a 1024^2 request and the 2048^2 request through all 8 blocks against the stored oracle rows
    check_deep_rows(run, out, "cfg5_mixed8", 0)
    check_deep_rows(run, out, "cfg5_mixed8", 5)
    # the 2048^2 request inside the packed batch, first block, sampled rows
    out1 = run.packed(n_blocks=1)
    r = 5
    L = wl.token_lens[r]
    rows = np.unique(np.concatenate([[0, 127, 128, L - 1], np.random.default_rng(1).integers(0, L, size=28)]))
    ref5 = O.block_forward(W.bf16_to_f64(wl.tokens[r]), W.bf16_to_f64(wl.cond[r]), f64w(wl.weights[0]),
                           wl.dims.n_heads, wl.dims.ln_eps, rows=rows)
    got5 = run.rows(out1, r).cpu().numpy().astype(np.float64)[rows]
    assert O.error_metric(got5, ref5) <= TOL
    run.close()


def test_cfg5_another_seeded_mix(B):
    """The mixed-resolution configuration drawn with another seed (another resolution mix, request order and
    set of packed offsets: 512, 512, 1024, 256, 1024, 1024, 256, 256): the last 512^2 and the last 256^2 request
    against the oracle through all 8 blocks, everything finite, packed == alone for one request of each
    resolution present."""
    wl = W.make_workload("cfg5_mixed8", seed=2)
    assert [q.height for q in wl.requests] == [512, 512, 1024, 256, 1024, 1024, 256, 256]
    run = DeviceRun(B, wl)
    out = run.packed()
    assert bool(run.torch.isfinite(out).all())
    ref = oracle_requests(wl, [1, 7])
    check_request(run, out, 1, ref[1])
    check_request(run, out, 7, ref[7])
    check_packed_equals_alone(run, out, requests=[1, 4, 7])
    run.close()


# ----------------------------------------------------------------------------- edge cases
@pytest.mark.parametrize("dims,reqs", [
    (W.LARGE, [(16, 16, 0)]),                                    # a single token: a = v
    (W.LARGE, [(176, 176, 6), (16, 16, 128), (16, 16, 0), (240, 320, 0)]),   # 127, 129, 1, 300 tokens
    (W.SMALL, [(256, 256, 3), (16, 16, 0), (128, 160, 49)]),     # head_dim 64, ragged
])
def test_ragged_lengths_one_block(B, dims, reqs):
    wl = W.make_custom("ragged", dims, 2, [(h, w, t) for (h, w, t) in reqs], seed=3)
    run = DeviceRun(B, wl)
    out = run.packed()
    ref = oracle_requests(wl, range(len(reqs)))
    for r in range(len(reqs)):
        check_request(run, out, r, ref[r])
    check_packed_equals_alone(run, out)
    run.close()


def test_sixty_four_requests(B):
    rng = np.random.default_rng(5)
    reqs = [(16, 16, int(rng.integers(0, 40))) for _ in range(64)]
    wl = W.make_custom("many", W.SMALL, 1, reqs, seed=4, timestep_cond=False)
    run = DeviceRun(B, wl, max_requests=64)
    out = run.packed()
    ref = oracle_requests(wl, range(64))
    for r in range(64):
        check_request(run, out, r, ref[r])
    check_packed_equals_alone(run, out, requests=[0, 17, 63])
    run.close()


def test_many_short_requests_in_a_long_batch(B):
    # 48 requests of 17..40 tokens: about a thousand packed rows, so the LayerNorm kernel that streams
    # rows through shared memory runs (it keeps one request's modulation vectors per CTA and must reload
    # them several times inside each CTA's chunk of rows), as do several GEMM row tiles that mix requests
    rng = np.random.default_rng(6)
    reqs = [(16 * int(rng.integers(1, 3)), 16 * int(rng.integers(1, 3)), int(rng.integers(13, 24))) for _ in range(48)]
    wl = W.make_custom("short", W.SMALL, 2, reqs, seed=6)
    assert wl.total_tokens > 4 * 148 + 100
    run = DeviceRun(B, wl, max_requests=48)
    out = run.packed()
    ref = oracle_requests(wl, range(48))
    for r in range(48):
        check_request(run, out, r, ref[r])
    check_packed_equals_alone(run, out, requests=[0, 23, 47])
    run.close()


def test_widest_hidden_size(B):
    # hidden 4096 (the largest the library takes): 16 KB rows leave one row buffer per warp in the
    # streaming LayerNorm kernel, and the GEMMs get a K that is not a multiple of 3072
    dims = W.ModelDims(hidden=4096, n_heads=32, head_dim=128, mlp_hidden=4096, cond_dim=256)
    wl = W.make_custom("wide", dims, 1, [(256, 256, 384), (64, 64, 0)], seed=8)
    assert wl.total_tokens >= 4 * 148
    run = DeviceRun(B, wl)
    out = run.packed()
    ref = oracle_requests(wl, [0, 1])
    check_request(run, out, 0, ref[0])
    check_request(run, out, 1, ref[1])
    check_packed_equals_alone(run, out)
    run.close()


@pytest.mark.parametrize("hidden,heads,head_dim,mlp,cond", [(64, 1, 64, 64, 1), (128, 1, 128, 64, 3), (192, 3, 64, 320, 5)])
def test_smallest_dimensions(B, hidden, heads, head_dim, mlp, cond):
    # the smallest shapes the library accepts: every GEMM is narrower than one 256-column tile and has one or a few
    # K steps, a single head, a cond vector of one to five channels
    dims = W.ModelDims(hidden=hidden, n_heads=heads, head_dim=head_dim, mlp_hidden=mlp, cond_dim=cond)
    wl = W.make_custom("tiny", dims, 2, [(32, 48, 3), (16, 16, 0), (160, 160, 31)], seed=17, timestep_cond=False)
    run = DeviceRun(B, wl)
    out = run.packed()
    ref = oracle_requests(wl, range(3))
    for r in range(3):
        check_request(run, out, r, ref[r])
    check_packed_equals_alone(run, out)
    run.close()


def test_zero_gate_returns_input_exactly(B):
    wl = W.make_custom("zerogate", W.SMALL, 2, [(256, 256, 5), (64, 64, 0)], seed=6, timestep_cond=False)
    H = wl.dims.hidden
    for w in wl.weights:
        for i in (2, 5):
            w["w_ada"][:, i * H:(i + 1) * H] = 0
            w["b_ada"][i * H:(i + 1) * H] = 0
    run = DeviceRun(B, wl)
    out = run.packed().cpu().numpy()
    np.testing.assert_array_equal(out, W.bf16_bits_to_f32(wl.packed_tokens()))
    run.close()


def test_row_permutation_equivariance(B):
    wl = W.make_custom("perm", W.SMALL, 1, [(256, 256, 44)], seed=7, timestep_cond=False)
    run = DeviceRun(B, wl)
    out = run.packed().cpu().numpy()
    perm = np.random.default_rng(0).permutation(wl.total_tokens)
    tokp = run.tok[run.torch.from_numpy(perm).cuda()].contiguous()
    outp = run.ctx.dit_step_forward(tokp, wl.token_lens, run.cond, 1).cpu().numpy()
    rms = float(np.sqrt(np.mean(out.astype(np.float64) ** 2)))
    assert np.abs(outp - out[perm]).max() / rms <= 2e-3      # same math, different key order in the softmax
    run.close()


def test_null_biases_mean_zero(B):
    wl = W.make_custom("nobias", W.SMALL, 1, [(128, 128, 9)], seed=8, timestep_cond=False)
    import torch
    ctx = B.context_for(wl.dims, 1, wl.total_tokens, 1)
    dev = {k: B.bits_to_cuda_bf16(v) for k, v in wl.weights[0].items() if k.startswith("w_")}
    ctx.dit_load_block_weights(0, dev)
    out = ctx.dit_step_forward(B.bits_to_cuda_bf16(wl.packed_tokens()), wl.token_lens, B.bits_to_cuda_bf16(wl.cond), 1)
    torch.cuda.synchronize()
    w = f64w(wl.weights[0])
    for k in w:
        if k.startswith("b_"):
            w[k] = np.zeros_like(w[k])
    ref = O.block_forward(W.bf16_to_f64(wl.tokens[0]), W.bf16_to_f64(wl.cond[0]), w, wl.dims.n_heads, wl.dims.ln_eps)
    assert O.error_metric(out.cpu().numpy(), ref) <= TOL
    ctx.close()


# ----------------------------------------------------------------------------- boundary behaviour on the device
def test_pack_tokens_and_host_entry_point(B):
    import torch
    wl = W.make_custom("pack", W.SMALL, 1, [(64, 64, 7), (16, 16, 0), (96, 32, 100)], seed=9, timestep_cond=False)
    run = DeviceRun(B, wl)
    per_req = [B.bits_to_cuda_bf16(t) for t in wl.tokens]
    packed = run.ctx.dit_pack_tokens(per_req)
    torch.cuda.synchronize()
    assert torch.equal(packed.view(torch.int16), run.tok.view(torch.int16))
    out = run.packed()
    h_tok = torch.from_numpy(wl.packed_tokens().view(np.int16)).pin_memory()
    h_cond = torch.from_numpy(wl.cond.view(np.int16)).pin_memory()
    h_out = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    run.ctx.dit_step_forward_host(h_tok, wl.token_lens, h_cond, 1, h_out)
    assert torch.equal(h_out, out.cpu())
    run.close()


def test_host_steps_two_in_flight(B):
    """dit_step_forward_host_async keeps two steps in flight: the tokens of step k + 1 go in under step k and
    the output of step k goes out under step k + 1.  Six steps alternate two different batches of the same shape
    through two host output buffers; every delivered output is bit-identical to the device-buffer step of its
    batch, whatever the copies overlapped with."""
    import torch
    wl_a = W.make_custom("pipe_a", W.LARGE, 2, [(512, 512, 96), (256, 256, 64)], seed=31)
    wl_b = W.make_custom("pipe_b", W.LARGE, 2, [(512, 512, 96), (256, 256, 64)], seed=32)
    run = DeviceRun(B, wl_a)                                   # both batches run on wl_a's weights
    want = []
    for wl in (wl_a, wl_b):
        out = run.ctx.dit_step_forward(B.bits_to_cuda_bf16(wl.packed_tokens()), wl.token_lens, B.bits_to_cuda_bf16(wl.cond), 2)
        torch.cuda.synchronize()
        want.append(out.cpu())
    assert not torch.equal(want[0], want[1])
    h_tok = [torch.from_numpy(wl.packed_tokens().view(np.int16)).pin_memory() for wl in (wl_a, wl_b)]
    h_cond = [torch.from_numpy(wl.cond.view(np.int16)).pin_memory() for wl in (wl_a, wl_b)]
    h_out = [torch.full(want[0].shape, float("nan"), dtype=torch.float32).pin_memory() for _ in range(2)]
    lens = wl_a.token_lens
    ctx = run.ctx
    ctx.dit_host_wait(0)                                       # nothing outstanding yet: returns at once
    ctx.dit_step_forward_host_async(h_tok[0], lens, h_cond[0], 2, h_out[0])
    for k in range(1, 6):
        ctx.dit_step_forward_host_async(h_tok[k & 1], lens, h_cond[k & 1], 2, h_out[k & 1])
        ctx.dit_host_wait(1)                                   # step k - 1 has arrived
        assert torch.equal(h_out[(k - 1) & 1], want[(k - 1) & 1]), f"step {k - 1}"
        h_out[(k - 1) & 1].fill_(float("nan"))                 # its buffer is free again for step k + 1
    ctx.dit_host_wait(0)
    assert torch.equal(h_out[1], want[1])
    with pytest.raises(B.DitError) as e:
        ctx.dit_host_wait(2)
    assert e.value.status == 1
    ctx.dit_ctx_poll_status()
    run.close()


def test_error_codes(B):
    import torch
    wl = W.make_custom("err", W.SMALL, 1, [(64, 64, 0)], seed=10, timestep_cond=False)
    ctx = B.context_for(wl.dims, 2, 64, 2)
    tok, cond = B.bits_to_cuda_bf16(wl.packed_tokens()), B.bits_to_cuda_bf16(wl.cond)
    with pytest.raises(B.DitError) as e:                       # nothing loaded yet
        ctx.dit_step_forward(tok[:16].contiguous(), [16], cond, 1)
    assert e.value.status == 4
    B.upload_weights(ctx, wl.weights)
    with pytest.raises(B.DitError) as e:                       # block 1 still missing
        ctx.dit_step_forward(tok[:16].contiguous(), [16], cond, 2)
    assert e.value.status == 4
    with pytest.raises(B.DitError) as e:                       # more tokens than max_total_tokens
        ctx.dit_step_forward(torch.cat([tok] * 5)[:65].contiguous(), [65], cond, 1)
    assert e.value.status == 3
    with pytest.raises(B.DitError) as e:                       # more blocks than slots
        ctx.dit_step_forward(tok[:16].contiguous(), [16], cond, 3)
    assert e.value.status == 3
    import ctypes as C
    lens = (C.c_int32 * 2)(16, 0)
    out = torch.empty((16, wl.dims.hidden), dtype=torch.float32, device="cuda")
    st = ctx.lib.dit_step_forward(ctx.handle, C.c_void_p(tok.data_ptr()), lens, 2, C.c_void_p(cond.data_ptr()), 1,
                                  C.c_void_p(out.data_ptr()), None)
    assert st == 1                                             # a zero-length request
    assert b"at least one token" in ctx.lib.dit_last_error(ctx.handle)
    out.fill_(7.0)
    st = ctx.lib.dit_step_forward(ctx.handle, None, None, 0, None, 1, None, None)
    assert st == 0                                             # empty batch: no-op
    torch.cuda.synchronize()
    assert float(out.min()) == 7.0
    ctx.dit_ctx_poll_status()
    ctx.close()


def test_bounded_wait_expiry_sets_the_status_word_once(B):
    """The failure path of every kernel: a bounded wait that runs out makes the kernel return and set
    the device status word.  A one-CTA test kernel waits (limit: tens of microseconds) on a barrier that
    nothing signals; the poll then reports the timeout once and the context keeps working."""
    wl = W.make_custom("expire", W.SMALL, 1, [(64, 64, 3)], seed=14, timestep_cond=False)
    run = DeviceRun(B, wl)
    want = run.packed()
    run.ctx.dit_ctx_poll_status()                      # clean before
    run.ctx.dit_debug_expire_wait()
    run.torch.cuda.synchronize()
    with pytest.raises(B.DitError) as e:
        run.ctx.dit_ctx_poll_status()
    assert e.value.status == 7 and "wait-expiry test" in str(e.value)      # DIT_ERR_TIMEOUT, names the kernel
    run.ctx.dit_ctx_poll_status()                      # reported once, then clear
    assert run.torch.equal(run.packed(), want)         # the context is still usable
    run.close()


def test_clock_probe_reports_plausible_clocks(B):
    """The measurement hook: attention CTAs of a 1024^2 request (36 key blocks) leave the SM clock they ran at and
    their cycles per key block, GEMM CTAs theirs; with the hook off nothing is written."""
    wl = W.make_custom("probe", W.LARGE, 1, [(1024, 1024, 512)], seed=16)
    run = DeviceRun(B, wl)
    assert run.ctx.dit_debug_clock_probe(True) == (0, 0, 0)
    run.packed()
    mhz, cyc, gemm_mhz = run.ctx.dit_debug_clock_probe(False)
    assert 500 <= mhz <= 2100 and 1500 <= cyc <= 8000 and 500 <= gemm_mhz <= 2100, (mhz, cyc, gemm_mhz)
    run.packed()
    assert run.ctx.dit_debug_clock_probe(False) == (0, 0, 0)
    run.close()


def test_poison_hook_makes_unwritten_reads_visible(B):
    """The poison fill itself: after it every activation tap reads as NaN and the guards are whole;
    damaging a guard by hand is reported."""
    import torch
    wl = W.make_custom("poison", W.SMALL, 1, [(64, 64, 3)], seed=15, timestep_cond=False)
    run = DeviceRun(B, wl)
    run.packed()
    run.ctx.dit_debug_poison()
    torch.cuda.synchronize()
    for name in ("h", "qkv", "attn", "u", "mod", "stream"):
        assert bool(torch.isnan(run.ctx.dit_debug_tap(name).float()).all()), name
    assert run.ctx.dit_debug_check_guards() == 0
    # the guard right after the residual stream region: clobber one word through a view of the workspace
    base = (run.ctx.workspace.data_ptr() + 1023) // 1024 * 1024 - run.ctx.workspace.data_ptr()
    import ctypes as C
    ptr, rows, cols, eb = C.c_void_p(), C.c_int64(), C.c_int64(), C.c_int32()
    assert run.ctx.lib.dit_debug_tap(run.ctx.handle, B.TAPS["h"], C.byref(ptr), C.byref(rows), C.byref(cols), C.byref(eb)) == 0
    h_off = ptr.value - run.ctx.workspace.data_ptr()
    assert h_off - 1024 >= base
    run.ctx.workspace[h_off - 1024:h_off - 1020] = 0           # last KiB before `h` is the stream's guard
    assert run.ctx.dit_debug_check_guards() == 1
    run.ctx.dit_debug_poison()                                 # rewrites the guards
    assert run.ctx.dit_debug_check_guards() == 0
    out = run.packed()
    assert bool(torch.isfinite(out).all())
    run.close()


def test_step_replays_from_a_cuda_graph(B):
    """The step neither allocates nor synchronises, so a caller can capture it once and replay it:
    this is what removes the launch overhead that dominates small-resolution steps (Section 3 of
    the paper motivates batching small requests with exactly that overhead)."""
    import torch
    wl = W.make_custom("graph", W.SMALL, 2, [(256, 256, 0), (64, 64, 9)], seed=12, timestep_cond=False)
    run = DeviceRun(B, wl)
    want = run.packed().clone()
    out = torch.zeros_like(want)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run.ctx.dit_step_forward(run.tok, wl.token_lens, run.cond, 2, out=out)     # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        run.ctx.dit_step_forward(run.tok, wl.token_lens, run.cond, 2, out=out)
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, want)
    # new token values in the same buffers: the replay follows them
    run.tok.copy_(run.tok.flip(0).contiguous())
    graph.replay()
    torch.cuda.synchronize()
    fresh = run.ctx.dit_step_forward(run.tok, wl.token_lens, run.cond, 2)
    torch.cuda.synchronize()
    assert torch.equal(out, fresh)
    run.ctx.dit_ctx_poll_status()
    run.close()


def test_two_contexts_on_two_streams_do_not_interfere(B):
    """Two contexts (different models, different batches) stepping at the same time on two streams,
    their launches interleaved by the host: each result is bit-identical to the one the context
    produces on its own.  The library keeps no state outside a context and its workspace, so
    contexts may be driven concurrently (only calls on ONE context must be serial)."""
    import torch
    wl_a = W.make_custom("ctx_a", W.SMALL, 2, [(256, 256, 7), (96, 64, 0), (64, 64, 3)], seed=31)
    wl_b = W.make_custom("ctx_b", W.LARGE, 1, [(128, 128, 16), (64, 96, 0)], seed=32)
    run_a, run_b = DeviceRun(B, wl_a), DeviceRun(B, wl_b)
    want_a, want_b = run_a.packed().clone(), run_b.packed().clone()
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    out_a = [torch.zeros_like(want_a) for _ in range(3)]
    out_b = [torch.zeros_like(want_b) for _ in range(3)]
    torch.cuda.synchronize()
    for i in range(3):
        run_a.ctx.dit_step_forward(run_a.tok, wl_a.token_lens, run_a.cond, run_a.nb, out=out_a[i], stream=sa)
        run_b.ctx.dit_step_forward(run_b.tok, wl_b.token_lens, run_b.cond, run_b.nb, out=out_b[i], stream=sb)
    torch.cuda.synchronize()
    run_a.ctx.dit_ctx_poll_status()
    run_b.ctx.dit_ctx_poll_status()
    for i in range(3):
        assert torch.equal(out_a[i], want_a), f"context A, step {i}"
        assert torch.equal(out_b[i], want_b), f"context B, step {i}"
    assert run_a.ctx.dit_debug_check_guards() == 0 and run_b.ctx.dit_debug_check_guards() == 0
    run_a.close()
    run_b.close()


@pytest.mark.parametrize("dims,length", [(W.SMALL, 600), (W.LARGE, 400)])
def test_growing_row_maximum_exercises_the_lazy_rescale(B, dims, length):
    """Q = K = 2h makes every query's own key its by far largest score (about 2^29 times the rest
    after exponentiation), so for rows beyond the first key tile the running maximum jumps in a
    later tile and the accumulator in tensor memory has to be rescaled: the rarely taken path."""
    n_text = length - 256
    wl = W.make_custom("selfmatch", dims, 1, [(256, 256, n_text)], seed=13, timestep_cond=False)
    H = dims.hidden
    wq = np.zeros((H, 3 * H), dtype=np.float32)
    idx = np.arange(H)
    wq[idx, idx] = 2.0
    wq[idx, H + idx] = 2.0
    wq[idx, 2 * H + idx] = 1.0
    wl.weights[0]["w_qkv"] = W.f32_to_bf16_bits(wq)
    wl.weights[0]["b_qkv"] = W.f32_to_bf16_bits(np.zeros(3 * H, dtype=np.float32))
    run = DeviceRun(B, wl)
    out = run.packed()
    taps = {0: {}}
    ref = oracle_requests(wl, [0], taps=taps)
    # the scores really are this peaked: the self key carries almost all of the weight
    qkv = taps[0]["qkv"]
    d = dims.head_dim
    s = (qkv[300, :d] @ qkv[:, H:H + d].T) / np.sqrt(d)
    assert s.argmax() == 300 and s[300] - np.partition(s, -2)[-2] > 8 * np.log(2.0) * 1.5
    got_a = run.ctx.dit_debug_tap("attn").cpu().numpy().astype(np.float64)
    assert O.error_metric(got_a, taps[0]["a"]) <= TOL
    check_request(run, out, 0, ref[0])
    assert run.torch.equal(out, run.packed())
    run.close()
