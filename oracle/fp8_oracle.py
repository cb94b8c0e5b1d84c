"""CPU oracle of the e4m3 mode in which ALL FOUR linear products of a block take 8-bit operands
(TEST INFRASTRUCTURE, not a product path; NumPy fp64, shares nothing with the CUDA path).

The mode is the last of the build's "next" rows (reduced-precision operands for the GEMMs; the paper
itself serves its models in 16-bit floating point, Section 6.1).  Each product is
`dit_oracle.fp8_linear`: every row of the left operand is scaled so that its largest magnitude maps to
448 and rounded to e4m3 (`dit_oracle.quantize_e4m3`), every column of the weight likewise, the product
of the quantised operands is exact and is scaled back.  The four left operands are the modulated
LayerNorm outputs (QKV projection, MLP up-projection), the attention output (output projection) and
the GELU output (MLP down-projection); for the parallel block form the concatenation [a | u] is one
operand with one scale per row.  Everything between the products (LayerNorm, modulation, attention,
GELU, gates, residuals) is the exact definition of `dit_oracle`.

Pins (tests/test_variant_oracle_pins.py): with every operand already on the e4m3 grid under
power-of-two scales the block equals the exact block; each product of the block equals
`fp8_linear` of the exact block's tap feeding it; the two-product form of `dit_oracle.block_forward`
(fp8=True) is recovered when the other two products are exact.
"""
from __future__ import annotations

from typing import Sequence

import numpy as np

from oracle import dit_oracle as O


def block_forward_fp8(x: np.ndarray, cond: np.ndarray, w, n_heads: int, eps: float, rows=None, taps=None,
                      positions=None, quantise=("qkv", "o", "fc1", "fc2")) -> np.ndarray:
    """The sequential adaLN-Zero block with the products named in `quantise` taken through fp8_linear."""
    H = x.shape[1]
    exact = lambda a, ww, bb: a @ ww + bb
    lin = {k: (O.fp8_linear if k in quantise else exact) for k in ("qkv", "o", "fc1", "fc2")}
    shift_a, scale_a, gate_a, shift_m, scale_m, gate_m = O.adaln_modulation(cond, w["w_ada"], w["b_ada"])
    h = O.modulate(O.layer_norm(x, eps), shift_a, scale_a)
    qkv = lin["qkv"](h, w["w_qkv"], w["b_qkv"])
    q, k, v = qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:]
    if "q_norm" in w:
        q = O.rms_norm_heads(q, w["q_norm"], n_heads, eps)
        k = O.rms_norm_heads(k, w["k_norm"], n_heads, eps)
    if positions is not None:
        q, k = O.rope_2d(q, positions, n_heads), O.rope_2d(k, positions, n_heads)
    a = O.attention(q, k, v, n_heads, rows)
    xr = x if rows is None else x[rows]
    x_mid = xr + gate_a * lin["o"](a, w["w_o"], w["b_o"])
    h2 = O.modulate(O.layer_norm(x_mid, eps), shift_m, scale_m)
    u = O.gelu_tanh(lin["fc1"](h2, w["w_fc1"], w["b_fc1"]))
    y = x_mid + gate_m * lin["fc2"](u, w["w_fc2"], w["b_fc2"])
    if taps is not None:
        taps.update(h1=h, qkv=np.concatenate([q, k, v], axis=1), a=a, x_mid=x_mid, h2=h2, u=u)
    return y


def parallel_block_forward_fp8(x: np.ndarray, cond: np.ndarray, w, n_heads: int, eps: float, rows=None, taps=None,
                               positions=None) -> np.ndarray:
    """The parallel block form with its three products (QKV, up-projection, output projection over [a | u])
    taken through fp8_linear; the concatenated row [a | u] gets one scale."""
    H = x.shape[1]
    shift, scale, gate = np.split(O.silu(cond) @ w["w_ada"] + w["b_ada"], 3)
    h = O.modulate(O.layer_norm(x, eps), shift, scale)
    qkv = O.fp8_linear(h, w["w_qkv"], w["b_qkv"])
    q, k, v = qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:]
    if "q_norm" in w:
        q = O.rms_norm_heads(q, w["q_norm"], n_heads, eps)
        k = O.rms_norm_heads(k, w["k_norm"], n_heads, eps)
    if positions is not None:
        q, k = O.rope_2d(q, positions, n_heads), O.rope_2d(k, positions, n_heads)
    a = O.attention(q, k, v, n_heads, rows)
    hr, xr = (h, x) if rows is None else (h[rows], x[rows])
    u = O.gelu_tanh(O.fp8_linear(hr, w["w_fc1"], w["b_fc1"]))
    y = xr + gate * O.fp8_linear(np.concatenate([a, u], axis=1), w["w_out"], w["b_out"])
    if taps is not None:
        taps.update(h1=h, qkv=np.concatenate([q, k, v], axis=1), a=a, u=u)
    return y


def stack_forward_fp8(x: np.ndarray, cond: np.ndarray, blocks: Sequence, n_heads: int, eps: float, positions=None) -> np.ndarray:
    """A stack of sequential / parallel blocks on one request, every product in e4m3."""
    for w in blocks:
        f = parallel_block_forward_fp8 if "w_out" in w else block_forward_fp8
        x = f(x, cond, w, n_heads, eps, positions=positions)
    return x


def step_forward_fp8(packed: np.ndarray, token_lens: Sequence[int], cond: np.ndarray, blocks: Sequence, n_heads: int,
                     eps: float, positions=None) -> np.ndarray:
    """One denoising step over a packed batch in the e4m3 mode: each request through the stack on its own."""
    out = np.empty_like(packed)
    p = 0
    for r, l in enumerate(token_lens):
        out[p:p + l] = stack_forward_fp8(packed[p:p + l], cond[r], blocks, n_heads, eps,
                                         None if positions is None else positions[r])
        p += l
    return out
