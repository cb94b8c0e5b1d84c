"""Range safety of the fp16-operand path and the bf16-operand mode (DIT_FLAG_BF16_OPERANDS).

The default path keeps fp16 operands inside (the benchmark configurations need fp16's 11 significant
bits to meet 1e-2).  The checkpoints the paper serves (its FLUX / SD3 class models, Section 6.1) are not
bound to fp16's range, so two things are checked here:

  * a value beyond +-65504 clamps instead of becoming infinite, and because masked attention
    probabilities are zeros multiplied by the NEXT request's value rows, one request's overflow must
    not reach its neighbours: they stay bit-identical to their alone runs and within the bar;
  * the bf16-operand mode computes the same step with bf16's range; its own bar against the same fp64
    oracle is BF16_TOL below (bf16 keeps 8 significant bits, so it cannot meet the fp16 path's 1e-2 at
    3072 wide; the measured values are printed).
"""
import numpy as np
import pytest

from oracle import dit_oracle as O
from paper_2510_01565_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = 1e-2          # the fp16-operand path's bar
BF16_TOL = 6e-2     # max|gpu - oracle| / rms(oracle) per request in the bf16-operand mode


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


def oracle_all(wl):
    return [O.stack_forward_alone(W.bf16_to_f64(wl.tokens[r]), W.bf16_to_f64(wl.cond[r]), [f64w(w) for w in wl.weights],
                                  wl.dims.n_heads, wl.dims.ln_eps) for r in range(len(wl.requests))]


def run_step(B, wl, flags=0, requests=None):
    import torch
    which = list(range(len(wl.requests))) if requests is None else requests
    lens = [wl.token_lens[r] for r in which]
    ctx = B.context_for(wl.dims, wl.n_blocks, sum(lens), len(which), flags=flags)
    B.upload_weights(ctx, wl.weights)
    tok = B.bits_to_cuda_bf16(np.concatenate([wl.tokens[r] for r in which], axis=0))
    cond = B.bits_to_cuda_bf16(wl.cond[which])
    ctx.dit_debug_poison()
    out = ctx.dit_step_forward(tok, lens, cond, wl.n_blocks)
    torch.cuda.synchronize()
    ctx.dit_ctx_poll_status()
    assert ctx.dit_debug_check_guards() == 0
    res, p = [], 0
    for l in lens:
        res.append(out[p:p + l].clone())
        p += l
    ctx.close()
    return res


@pytest.mark.parametrize("dims,reqs,nb", [
    (W.SMALL, [(128, 128, 7), (256, 256, 0), (16, 16, 40)], 2),
    (W.LARGE, [(256, 256, 77), (512, 512, 512)], 2),
])
def test_bf16_operand_mode_against_the_oracle(B, dims, reqs, nb):
    wl = W.make_custom("bf16", dims, nb, reqs, seed=21)
    ref = oracle_all(wl)
    got16 = run_step(B, wl)
    gotbf = run_step(B, wl, flags=B.DIT_FLAG_BF16_OPERANDS)
    for r in range(len(reqs)):
        e16 = O.error_metric(got16[r].cpu().numpy(), ref[r])
        ebf = O.error_metric(gotbf[r].cpu().numpy(), ref[r])
        print(f"hidden {dims.hidden} request {r}: max|d|/rms fp16 operands {e16:.3e}, bf16 operands {ebf:.3e}")
        assert e16 <= TOL
        assert ebf <= BF16_TOL
        assert ebf > e16                       # the mode really ran with the coarser operands
    # packed == alone holds in this mode too
    alone = run_step(B, wl, flags=B.DIT_FLAG_BF16_OPERANDS, requests=[1])
    import torch
    assert torch.equal(alone[0], gotbf[1])


def test_bf16_mode_parallel_blocks_and_taps(B):
    import torch
    wl = W.make_custom("bf16par", W.SMALL, 2, [(128, 128, 9), (64, 64, 0)], seed=22)
    rng = np.random.default_rng(22)
    wl.weights = [wl.weights[0], W.draw_parallel_block_weights(rng, wl.dims)]
    ref = oracle_all(wl)
    got = run_step(B, wl, flags=B.DIT_FLAG_BF16_OPERANDS)
    for r in range(2):
        assert O.error_metric(got[r].cpu().numpy(), ref[r]) <= BF16_TOL
    # the 16-bit intermediates are bf16 in this mode: q/k/v of a one-block run against the oracle's
    wl1 = W.make_custom("bf16tap", W.SMALL, 1, [(128, 128, 9)], seed=23)
    ctx = B.context_for(wl1.dims, 1, wl1.total_tokens, 1, flags=B.DIT_FLAG_BF16_OPERANDS)
    B.upload_weights(ctx, wl1.weights)
    ctx.dit_step_forward(B.bits_to_cuda_bf16(wl1.packed_tokens()), wl1.token_lens, B.bits_to_cuda_bf16(wl1.cond), 1)
    torch.cuda.synchronize()
    taps = {}
    O.block_forward(W.bf16_to_f64(wl1.tokens[0]), W.bf16_to_f64(wl1.cond[0]), f64w(wl1.weights[0]), wl1.dims.n_heads,
                    wl1.dims.ln_eps, taps=taps)
    qkv = ctx.dit_debug_tap("qkv")
    assert qkv.dtype == torch.bfloat16
    assert O.error_metric(qkv.float().cpu().numpy(), taps["qkv"]) <= BF16_TOL
    ctx.close()


def test_bf16_mode_refuses_what_it_was_not_built_for(B):
    wl = W.make_custom("bf16err", W.SMALL, 2, [(64, 64, 3)], seed=24)
    for extra in (B.DIT_FLAG_QK_RMSNORM, B.DIT_FLAG_ROPE_2D, B.DIT_FLAG_FP8_GEMM):
        with pytest.raises(B.DitError) as e:
            B.context_for(wl.dims, 2, 64, 1, flags=B.DIT_FLAG_BF16_OPERANDS | extra)
        assert e.value.status == 2
    ctx = B.context_for(wl.dims, 2, 64, 1, flags=B.DIT_FLAG_BF16_OPERANDS)
    dev = {k: B.bits_to_cuda_bf16(v) for k, v in wl.weights[0].items()}
    with pytest.raises(B.DitError) as e:
        ctx.dit_load_dual_block_weights(0, dev, dev)
    assert e.value.status == 2
    ctx.close()


def test_overflow_in_one_request_stays_in_that_request(B):
    """Request 1's conditioning vector is scaled by 2^20: its modulation scale, and with it h, q, k, v
    and u, leave fp16's range.  The fp16 path must write clamped finite values, and requests 0 and 2
    (whose masked-out probabilities multiply request 1's rows inside shared key tiles) must come out
    bit-identical to their alone runs and within the bar."""
    import torch
    wl = W.make_custom("overflow", W.SMALL, 2, [(160, 160, 17), (96, 96, 30), (128, 64, 5)], seed=25, timestep_cond=False)
    big = W.bf16_bits_to_f32(wl.cond[1]) * np.float32(2.0 ** 20)
    wl.cond[1] = W.f32_to_bf16_bits(big)
    packed = run_step(B, wl)
    for r in range(3):
        assert bool(torch.isfinite(packed[r]).all()), f"request {r} holds a non-finite value"
    # the overflow really happens: in the oracle, request 1's q/k/v leave fp16's range in block 0
    taps = {}
    O.block_forward(W.bf16_to_f64(wl.tokens[1]), W.bf16_to_f64(wl.cond[1]), f64w(wl.weights[0]), wl.dims.n_heads,
                    wl.dims.ln_eps, taps=taps)
    assert np.abs(taps["qkv"]).max() > 65504.0 and np.abs(taps["h1"]).max() > 65504.0
    for r in (0, 2):
        alone = run_step(B, wl, requests=[r])
        assert torch.equal(alone[0], packed[r]), f"request {r} changed next to an overflowing request"
        ref = O.stack_forward_alone(W.bf16_to_f64(wl.tokens[r]), W.bf16_to_f64(wl.cond[r]), [f64w(w) for w in wl.weights],
                                    wl.dims.n_heads, wl.dims.ln_eps)
        assert O.error_metric(packed[r].cpu().numpy(), ref) <= TOL


def test_bf16_mode_holds_activations_beyond_fp16_range(B):
    """W_fc1 and b_fc1 scaled by 2^19, W_fc2 by 2^-19: the MLP's hidden activation u reaches about 1e5
    while the block's result is unchanged in exact arithmetic.  The bf16-operand mode meets its bar on
    these inputs; the fp16 path clamps u (finite, but far from the oracle), which is what the mode is for."""
    import torch
    s = np.float32(2.0 ** 19)
    wl = W.make_custom("wide_range", W.SMALL, 2, [(128, 128, 7), (64, 96, 0)], seed=26)
    for w in wl.weights:
        w["w_fc1"] = W.f32_to_bf16_bits(W.bf16_bits_to_f32(w["w_fc1"]) * s)       # exact: a power of two
        w["b_fc1"] = W.f32_to_bf16_bits(W.bf16_bits_to_f32(w["b_fc1"]) * s)
        w["w_fc2"] = W.f32_to_bf16_bits(W.bf16_bits_to_f32(w["w_fc2"]) / s)
    ref = oracle_all(wl)
    taps = {}
    O.block_forward(W.bf16_to_f64(wl.tokens[0]), W.bf16_to_f64(wl.cond[0]), f64w(wl.weights[0]), wl.dims.n_heads,
                    wl.dims.ln_eps, taps=taps)
    assert np.abs(taps["u"]).max() > 65504.0
    gotbf = run_step(B, wl, flags=B.DIT_FLAG_BF16_OPERANDS)
    got16 = run_step(B, wl)
    for r in range(2):
        ebf = O.error_metric(gotbf[r].cpu().numpy(), ref[r])
        e16 = O.error_metric(got16[r].cpu().numpy(), ref[r])
        print(f"request {r}: bf16 operands {ebf:.3e}; fp16 operands (clamped) {e16:.3e}")
        assert ebf <= BF16_TOL
        assert bool(torch.isfinite(got16[r]).all())
        assert e16 > BF16_TOL                  # the default path cannot represent these activations
