"""The allocation-free modulation entry point against the context path (collected last on purpose).

Some hosts of this library may not allocate device memory at all: a plugin that runs inside another
runtime's execution phase, or a process whose GPU memory pool is owned by a framework and handed
out as fixed buffers.  `dit_modulation_noalloc` serves them: it takes only caller buffers and
keeps its one piece of scratch (the fp32 bias) in a fixed array inside the library.  This test calls
it through the C ABI twice in a row with different inputs and compares each result with the `mod`
vectors that `dit_step_forward` computes for the same block, and with the CPU oracle's.
"""
import numpy as np
import pytest

from oracle import dit_oracle as O
from paper_2510_01565_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = 1e-5   # same bound the parity tests put on the modulation vectors (max|d| / rms)


def _rel(got, ref):
    ref = ref.astype(np.float64)
    return float(np.abs(got.astype(np.float64) - ref).max() / np.sqrt(np.mean(ref ** 2)))


def test_noalloc_modulation_matches_context_path_twice():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    from paper_2510_01565_b200 import binding as B, build
    build.build_library()

    wl = W.make_custom("noalloc", W.SMALL, 2, [(64, 64, 3), (32, 48, 0), (16, 16, 9)], seed=11)
    H, R = wl.dims.hidden, len(wl.requests)
    tok, cond = B.bits_to_cuda_bf16(wl.packed_tokens()), B.bits_to_cuda_bf16(wl.cond)

    # existing path: block 1 loaded WITHOUT its modulation bias, so the second no-alloc call below
    # must have cleared the bias the first call left in the shared scratch
    ctx = B.context_for(wl.dims, 2, wl.total_tokens, R)
    dev = [{k: B.bits_to_cuda_bf16(v) for k, v in w.items()} for w in wl.weights]
    ctx.dit_load_block_weights(0, dev[0])
    ctx.dit_load_block_weights(1, {k: v for k, v in dev[1].items() if k != "b_ada"})
    ctx.dit_step_forward(tok, wl.token_lens, cond, 2)
    torch.cuda.synchronize()
    ref = ctx.dit_debug_tap("mod").cpu().numpy().reshape(R, 2, 6 * H)

    out = torch.full((R, 6 * H), float("nan"), dtype=torch.float32, device="cuda")
    B.dit_modulation_noalloc(cond, dev[0]["w_ada"], dev[0]["b_ada"], out)          # call 1: with bias
    torch.cuda.synchronize()
    got0 = out.cpu().numpy()
    out.fill_(float("nan"))
    B.dit_modulation_noalloc(cond, dev[1]["w_ada"], None, out)                     # call 2: NULL bias
    torch.cuda.synchronize()
    got1 = out.cpu().numpy()

    assert np.isfinite(got0).all() and np.isfinite(got1).all()
    assert _rel(got0, ref[:, 0]) <= TOL
    assert _rel(got1, ref[:, 1]) <= TOL
    assert np.abs(got0 - got1).max() > 1e-3        # the two calls really computed different blocks
    # and directly against the oracle's modulation vectors (block 1 without its bias)
    for r in range(R):
        c = W.bf16_to_f64(wl.cond[r])
        w0, w1 = ({k: W.bf16_to_f64(v) for k, v in wl.weights[b].items()} for b in (0, 1))
        want0 = np.concatenate(O.adaln_modulation(c, w0["w_ada"], w0["b_ada"]))
        want1 = np.concatenate(O.adaln_modulation(c, w1["w_ada"], np.zeros_like(w1["b_ada"])))
        assert _rel(got0[r], want0) <= TOL
        assert _rel(got1[r], want1) <= TOL
    ctx.close()


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    import ctypes as C
    import torch
    from paper_2510_01565_b200 import binding as B
    lib = B.load_library()
    buf = torch.zeros(64, dtype=torch.float32, device="cuda")
    p = C.c_void_p(buf.data_ptr())
    assert lib.dit_modulation_noalloc(p, p, None, 1, 64, 8192, p, None) == 3       # hidden beyond the scratch
    assert lib.dit_modulation_noalloc(p, p, None, 1, 5000, 64, p, None) == 3       # cond_dim beyond the limit
    assert lib.dit_modulation_noalloc(p, p, None, 65, 64, 64, p, None) == 3        # too many requests
    assert lib.dit_modulation_noalloc(p, p, None, 1, 64, 100, p, None) == 2        # unsupported hidden
    assert lib.dit_modulation_noalloc(None, p, None, 1, 64, 64, p, None) == 1
    assert lib.dit_modulation_noalloc(None, None, None, 0, 64, 64, None, None) == 0
    # W_ada is read with 16-byte loads: a view that starts 2 bytes into a buffer is refused on the host
    odd = C.c_void_p(buf.data_ptr() + 2)
    assert lib.dit_modulation_noalloc(p, odd, None, 1, 64, 64, p, None) == 1
    assert lib.dit_modulation_noalloc(p, p, None, 1, 64, 64, odd, None) == 1       # fp32 output at an odd half-word
    torch.cuda.synchronize()
    assert float(buf.abs().max()) == 0.0           # nothing was launched by the rejected calls
