"""CPU oracle for the shell around the block stack (TEST INFRASTRUCTURE, not a product path).

A full denoising step of a request, as the paper's serving system dispatches
it (Section 4: the latent of a request is carried from step to step and only
that latent moves between workers; Section 2: a step runs the transformer over
the request's whole latent): latent -> tokens, timestep -> conditioning
vector, the block stack (oracle/dit_oracle.py), tokens -> velocity, and the
sampler's update of the latent.  The paper runs these parts through PyTorch
model code and does not restate them; the forms below are the standard ones of
the latent DiT family it serves, with these readings:

  * latent z [16, h/8, w/8] for an h x w pixel request; 2 x 2 patches, so one
    token per 16 x 16 pixels (Section 6.1 token rule); a patch is flattened in
    (channel, dy, dx) order into 64 numbers;
  * token = patch W_in + b_in + pos(py, px), where pos is the fixed 2-D
    sine/cosine embedding: the first H/2 channels encode the patch row, the
    last H/2 the patch column; each half is [sin(p w_k) | cos(p w_k)] with
    w_k = 10000^(-k / (H/4)), k < H/4;
  * text tokens arrive already projected to H channels (the text encoder is
    outside the step) and follow the image tokens of their request;
  * tokens enter the block stack rounded to bf16 (the stack's input type);
  * conditioning: e(t) = [cos(t f_k) | sin(t f_k)], f_k = 10000^(-k/128),
    k < 128;  c = SiLU(e W_t1 + b_t1) W_t2 + b_t2 + pooled, rounded to bf16
    (the stack's conditioning type);
  * final layer: (shift, scale) = SiLU(c) W_fa + b_fa (H each);
    y = LN(x) (1 + scale) + shift;  v_tok = y W_out + b_out (64 per image
    token); text tokens produce no output; un-patchify v_tok into v shaped
    like z;
  * sampler: one explicit Euler step of the rectified-flow ODE,
    z <- z + (sigma_next - sigma_cur) v.

Everything is fp64 NumPy except the two stated roundings to bf16.  It shares
no code with the CUDA path and imports neither it nor torch.

Parity pins (tests/test_oracle_pins.py): patchify against independent index
arithmetic and as the inverse of unpatchify; sine/cosine embeddings at zero
and their unit-circle identity; embed / final layer with selector weights
(reduce to the patch, to LayerNorm); Euler against the closed-form solution
of the straight-line flow; a zero-initialised output layer moves the latent
by dsigma * b_out.
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence, Tuple

import numpy as np

from . import dit_oracle as blocks

LATENT_CHANNELS = 16
VAE_FACTOR = 8
PATCH = 2
PATCH_DIM = LATENT_CHANNELS * PATCH * PATCH   # 64
T_EMB_DIM = 256

ShellWeights = Dict[str, np.ndarray]


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of fp64 values to bf16, returned as fp64 (via fp32 first)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16 << 16
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


def latent_shape(height: int, width: int) -> Tuple[int, int, int]:
    return LATENT_CHANNELS, height // VAE_FACTOR, width // VAE_FACTOR


def patchify(z: np.ndarray) -> np.ndarray:
    """z [16, h8, w8] -> [gh*gw, 64]; token (py, px) in row-major order, patch in (c, dy, dx) order."""
    c, h8, w8 = z.shape
    gh, gw = h8 // PATCH, w8 // PATCH
    p = z.reshape(c, gh, PATCH, gw, PATCH)          # c, py, dy, px, dx
    p = p.transpose(1, 3, 0, 2, 4)                   # py, px, c, dy, dx
    return p.reshape(gh * gw, c * PATCH * PATCH)


def unpatchify(tok: np.ndarray, h8: int, w8: int) -> np.ndarray:
    gh, gw = h8 // PATCH, w8 // PATCH
    p = tok.reshape(gh, gw, LATENT_CHANNELS, PATCH, PATCH)
    p = p.transpose(2, 0, 3, 1, 4)                   # c, py, dy, px, dx
    return p.reshape(LATENT_CHANNELS, h8, w8)


def axis_embedding(pos: np.ndarray, dim: int) -> np.ndarray:
    """[len(pos), dim]: sin half then cos half, frequencies 10000^(-k/(dim/2))."""
    half = dim // 2
    omega = 10000.0 ** (-np.arange(half, dtype=np.float64) / half)
    arg = pos[:, None].astype(np.float64) * omega[None, :]
    return np.concatenate([np.sin(arg), np.cos(arg)], axis=1)


def pos_embed_2d(gh: int, gw: int, hidden: int) -> np.ndarray:
    """[gh*gw, hidden]: first half from the patch row, second half from the patch column."""
    py, px = np.meshgrid(np.arange(gh), np.arange(gw), indexing="ij")
    return np.concatenate([axis_embedding(py.reshape(-1), hidden // 2),
                           axis_embedding(px.reshape(-1), hidden // 2)], axis=1)


def embed_latent(z: np.ndarray, w: ShellWeights, hidden: int) -> np.ndarray:
    """Image tokens of one request, before the rounding to bf16."""
    _, h8, w8 = z.shape
    return patchify(z) @ w["w_in"] + w["b_in"] + pos_embed_2d(h8 // PATCH, w8 // PATCH, hidden)


def timestep_embedding(t: float) -> np.ndarray:
    half = T_EMB_DIM // 2
    f = 10000.0 ** (-np.arange(half, dtype=np.float64) / half)
    return np.concatenate([np.cos(t * f), np.sin(t * f)])


def timestep_cond(t: float, pooled: np.ndarray | None, w: ShellWeights) -> np.ndarray:
    """Conditioning vector of one request, before the rounding to bf16."""
    hdn = blocks.silu(timestep_embedding(t) @ w["w_t1"] + w["b_t1"])
    c = hdn @ w["w_t2"] + w["b_t2"]
    return c if pooled is None else c + pooled


def final_layer(x_img: np.ndarray, cond: np.ndarray, w: ShellWeights, eps: float) -> np.ndarray:
    """x_img [n_img, H] (image rows of one request), cond [C] -> v_tok [n_img, 64]."""
    hidden = x_img.shape[1]
    m = blocks.silu(cond) @ w["w_fa"] + w["b_fa"]
    shift, scale = m[:hidden], m[hidden:]
    y = blocks.modulate(blocks.layer_norm(x_img, eps), shift, scale)
    return y @ w["w_out"] + w["b_out"]


def euler_update(z: np.ndarray, v: np.ndarray, dsigma: float) -> np.ndarray:
    return z + dsigma * v


def denoise_step(latents: Sequence[np.ndarray], texts: Sequence[np.ndarray], timesteps: Sequence[float],
                 dsigmas: Sequence[float], pooled: Sequence[np.ndarray | None], shell: ShellWeights,
                 block_ws: Sequence[blocks.Weights], n_heads: int, eps: float, rope: bool = False):
    """One full step of every request (each on its own).  Returns (new latents, velocities, taps).

    texts[r] is [n_text_r, H] (already bf16-representable) or an empty array.
    taps holds the intermediate results the parity tests compare: cond (bf16-rounded), tokens
    (bf16-rounded, image then text rows) and the stack output, per request.  With `rope` the blocks
    apply the 2-D rotary term at the tokens' patch positions (RMS-norm of queries and keys is
    switched on by the block weights holding q_norm / k_norm).
    """
    new_latents, velocities, taps = [], [], []
    for z, txt, t, ds, pl in zip(latents, texts, timesteps, dsigmas, pooled):
        hidden = shell["w_in"].shape[1]
        cond = round_to_bf16(timestep_cond(t, pl, shell))
        img = round_to_bf16(embed_latent(z, shell, hidden))
        tokens = img if txt.shape[0] == 0 else np.concatenate([img, txt], axis=0)
        pos = blocks.patch_positions(z.shape[1] * VAE_FACTOR, z.shape[2] * VAE_FACTOR, txt.shape[0]) if rope else None
        x = blocks.stack_forward_alone(tokens, cond, block_ws, n_heads, eps, positions=pos, n_img=img.shape[0])
        v_tok = final_layer(x[:img.shape[0]], cond, shell, eps)
        v = unpatchify(v_tok, z.shape[1], z.shape[2])
        new_latents.append(euler_update(z, v, ds))
        velocities.append(v)
        taps.append({"cond": cond, "tokens": tokens, "x": x})
    return new_latents, velocities, taps
