"""Seeded synthetic inputs shaped like the paper's DiT serving workloads.

This module only *draws inputs*: request lists, token buffers, conditioning
vectors and block weights.  It holds none of the block's arithmetic and imports
neither the CUDA binding nor the CPU oracle, so that both sides can be fed the
same arrays.

Shapes follow the paper's workload description: four image resolutions
256^2 .. 2048^2 whose latent token counts are (H*W)/16^2 (Table 1 and the
"Workload and Dataset" paragraph of Section 6.1), a FLUX-like 3072-wide block
with 24 heads of 128 and 512 text tokens per prompt.  The paper's trained
weights and its prompt dataset are not needed for a step's cost or numerics;
N(0,1) tokens and N(0,0.02) weights stand in for them.

Every array the GPU sees is bf16.  Values are drawn in fp32, rounded once to
bf16 (round to nearest even) and kept as uint16 bit patterns; `bf16_to_f64`
widens those bits exactly for the oracle.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Sequence, Tuple

import numpy as np

PATCH_PIXELS = 16  # 8x VAE downsampling times patch size 2 (Section 6.1)
RESOLUTIONS = (256, 512, 1024, 2048)
MIX_WEIGHTS = (0.2, 0.35, 0.3, 0.15)

WEIGHT_NAMES = ("w_ada", "b_ada", "w_qkv", "b_qkv", "w_o", "b_o",
                "w_fc1", "b_fc1", "w_fc2", "b_fc2")


# --------------------------------------------------------------------------
# bf16 <-> numpy helpers (representation only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (nearest, ties to even); return uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp64 exactly."""
    return bf16_bits_to_f32(bits).astype(np.float64)


# --------------------------------------------------------------------------
# model / workload description
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class ModelDims:
    hidden: int
    n_heads: int
    head_dim: int
    mlp_hidden: int
    cond_dim: int
    ln_eps: float = 1e-6


@dataclass(frozen=True)
class Request:
    height: int
    width: int
    n_text_tokens: int
    timestep: float
    step_index: int = 0

    @property
    def n_image_tokens(self) -> int:
        return (self.height // PATCH_PIXELS) * (self.width // PATCH_PIXELS)

    @property
    def n_tokens(self) -> int:
        return self.n_image_tokens + self.n_text_tokens


@dataclass
class Workload:
    name: str
    dims: ModelDims
    n_blocks: int
    requests: List[Request]
    tokens: List[np.ndarray]            # per request [L_r, H] uint16 (bf16 bits)
    cond: np.ndarray                    # [R, C] uint16 (bf16 bits)
    weights: List[Dict[str, np.ndarray]] = field(default_factory=list)  # per block, bf16 bits

    @property
    def token_lens(self) -> List[int]:
        return [r.n_tokens for r in self.requests]

    @property
    def total_tokens(self) -> int:
        return sum(self.token_lens)

    @property
    def image_tokens(self) -> int:
        return sum(r.n_image_tokens for r in self.requests)

    def packed_tokens(self) -> np.ndarray:
        return np.concatenate(self.tokens, axis=0)

    def flops_per_step(self, n_blocks: int | None = None) -> float:
        """Algorithmic FLOPs: four GEMMs + block-diagonal attention per block."""
        nb = self.n_blocks if n_blocks is None else n_blocks
        h, f = self.dims.hidden, self.dims.mlp_hidden
        t = self.total_tokens
        lin = 2.0 * t * (h * 3 * h + h * h + 2 * h * f)
        att = 4.0 * h * sum(l * l for l in self.token_lens)
        return nb * (lin + att)


SMALL = ModelDims(hidden=384, n_heads=6, head_dim=64, mlp_hidden=1536, cond_dim=384)
LARGE = ModelDims(hidden=3072, n_heads=24, head_dim=128, mlp_hidden=12288, cond_dim=3072)

# name -> (dims, n_blocks, list of (resolution, n_text) or None for the seeded mix)
CONFIGS: Dict[str, Tuple[ModelDims, int, object]] = {
    "cfg1_small_256": (SMALL, 1, [(256, 0)]),
    "cfg2_512": (LARGE, 4, [(512, 512)]),
    "cfg3_1024x2": (LARGE, 4, [(1024, 512), (1024, 512)]),
    "cfg4_2048": (LARGE, 4, [(2048, 512)]),
    "cfg5_mixed8": (LARGE, 8, None),
}


def timestep_embedding(t: float, dim: int) -> np.ndarray:
    """Sinusoidal embedding of a real timestep: cos half then sin half (fp64)."""
    half = dim // 2
    freqs = np.exp(-math.log(10000.0) * np.arange(half, dtype=np.float64) / half)
    return np.concatenate([np.cos(t * freqs), np.sin(t * freqs)])


def draw_mixed_resolutions(rng: np.random.Generator, n: int) -> List[int]:
    idx = rng.choice(len(RESOLUTIONS), size=n, p=MIX_WEIGHTS)
    return [RESOLUTIONS[i] for i in idx]


def _normal_bf16(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return f32_to_bf16_bits(x)


def draw_block_weights(rng: np.random.Generator, dims: ModelDims, std: float = 0.02) -> Dict[str, np.ndarray]:
    """One block's ten tensors, row-major [in, out], bf16 bits, fixed draw order."""
    h, f, c = dims.hidden, dims.mlp_hidden, dims.cond_dim
    shapes = {"w_ada": (c, 6 * h), "b_ada": (6 * h,), "w_qkv": (h, 3 * h), "b_qkv": (3 * h,),
              "w_o": (h, h), "b_o": (h,), "w_fc1": (h, f), "b_fc1": (f,),
              "w_fc2": (f, h), "b_fc2": (h,)}
    return {k: _normal_bf16(rng, shapes[k], std) for k in WEIGHT_NAMES}


PARALLEL_WEIGHT_NAMES = ("w_ada", "b_ada", "w_qkv", "b_qkv", "w_fc1", "b_fc1", "w_out", "b_out")


def draw_parallel_block_weights(rng: np.random.Generator, dims: ModelDims, std: float = 0.02) -> Dict[str, np.ndarray]:
    """One parallel-form block's eight tensors, row-major [in, out], bf16 bits, fixed draw order."""
    h, f, c = dims.hidden, dims.mlp_hidden, dims.cond_dim
    shapes = {"w_ada": (c, 3 * h), "b_ada": (3 * h,), "w_qkv": (h, 3 * h), "b_qkv": (3 * h,),
              "w_fc1": (h, f), "b_fc1": (f,), "w_out": (h + f, h), "b_out": (h,)}
    return {k: _normal_bf16(rng, shapes[k], std) for k in PARALLEL_WEIGHT_NAMES}


def draw_qk_norm(rng: np.random.Generator, dims: ModelDims) -> Dict[str, np.ndarray]:
    """RMS-norm scales of the queries and keys, [head_dim] each, 1 + 0.1 N(0,1), bf16 bits.
    Drawn from a generator of their own so that the ten block tensors keep their draw order."""
    return {k: f32_to_bf16_bits(1.0 + 0.1 * rng.standard_normal(size=dims.head_dim, dtype=np.float32))
            for k in ("q_norm", "k_norm")}


def make_custom(name: str, dims: ModelDims, n_blocks: int,
                reqs: Sequence[Tuple[int, int, int]], seed: int = 0,
                timestep_cond: bool = True, with_weights: bool = True) -> Workload:
    """Workload from explicit (height, width, n_text) triples.

    Draw order from one generator: per request (t, tokens, pooled vector), then
    per block the ten weight tensors in WEIGHT_NAMES order.
    """
    rng = np.random.default_rng(seed)
    return _draw(name, dims, n_blocks, list(reqs), rng, timestep_cond, with_weights)


def _draw(name, dims, n_blocks, reqs, rng, timestep_cond, with_weights) -> Workload:
    requests, tokens, conds = [], [], []
    for (hh, ww, n_text) in reqs:
        t = float(rng.uniform(0.0, 1000.0))
        req = Request(hh, ww, n_text, t)
        tok = _normal_bf16(rng, (req.n_tokens, dims.hidden), 1.0)
        pooled = rng.standard_normal(size=dims.cond_dim, dtype=np.float32).astype(np.float64)
        if timestep_cond:
            c = timestep_embedding(t, dims.cond_dim) + pooled
        else:
            c = pooled
        requests.append(req)
        tokens.append(tok)
        conds.append(f32_to_bf16_bits(c.astype(np.float32)))
    weights = [draw_block_weights(rng, dims) for _ in range(n_blocks)] if with_weights else []
    return Workload(name, dims, n_blocks, requests, tokens, np.stack(conds), weights)


def make_workload(name: str, seed: int = 0, n_blocks: int | None = None,
                  with_weights: bool = True, n_blocks_drawn: int | None = None) -> Workload:
    """One of the five benchmark configurations, fully seeded.

    `n_blocks_drawn` draws only the first few blocks' weights (they come last in the draw order,
    so the requests, tokens, cond vectors and those blocks are unchanged) while `n_blocks` keeps
    the configuration's depth.
    """
    dims, nb, reqs = CONFIGS[name]
    nb = nb if n_blocks is None else n_blocks
    rng = np.random.default_rng(seed)
    if reqs is None:
        res = draw_mixed_resolutions(rng, 8)
        reqs = [(r, 512) for r in res]
    reqs3 = [(r, r, n_text) for (r, n_text) in reqs]
    # config 1 draws its cond vector directly; the large configs add a timestep embedding
    wl = _draw(name, dims, nb if n_blocks_drawn is None else min(nb, n_blocks_drawn), reqs3, rng,
               timestep_cond=(dims is LARGE), with_weights=with_weights)
    wl.n_blocks = nb
    return wl


# --------------------------------------------------------------------------
# inputs of a full denoising step (latent in, latent out) around the block stack
# --------------------------------------------------------------------------
LATENT_CHANNELS = 16     # latent z of an h x w request is [16, h/8, w/8] fp32
VAE_FACTOR = 8
PATCH_DIM = 64           # 16 channels x 2 x 2
T_EMB_DIM = 256

SHELL_WEIGHT_NAMES = ("w_in", "b_in", "w_t1", "b_t1", "w_t2", "b_t2", "w_fa", "b_fa", "w_out", "b_out")


def draw_shell_weights(rng: np.random.Generator, dims: ModelDims) -> Dict[str, np.ndarray]:
    """Embedding, timestep-MLP and final-layer tensors, row-major [in, out], bf16 bits.

    The patch embedding is drawn at 1/sqrt(64) so that tokens come out at unit scale like the
    N(0,1) token buffers of the step-only workloads; the rest at the 0.02 of the block weights.
    """
    h, c = dims.hidden, dims.cond_dim
    shapes = {"w_in": (PATCH_DIM, h), "b_in": (h,), "w_t1": (T_EMB_DIM, c), "b_t1": (c,),
              "w_t2": (c, c), "b_t2": (c,), "w_fa": (c, 2 * h), "b_fa": (2 * h,),
              "w_out": (h, PATCH_DIM), "b_out": (PATCH_DIM,)}
    return {k: _normal_bf16(rng, shapes[k], 0.125 if k == "w_in" else 0.02) for k in SHELL_WEIGHT_NAMES}


@dataclass
class StepInputs:
    """Per-request inputs of full denoising steps, plus the model's tensors."""
    dims: ModelDims
    requests: List[Request]
    latents: List[np.ndarray]          # per request [16, h/8, w/8] fp32, N(0,1)
    texts: List[np.ndarray]            # per request [n_text, H] uint16 (bf16 bits), N(0,1)
    pooled: np.ndarray                 # [R, C] fp32, N(0,1) (the prompt's pooled vector)
    dsigmas: np.ndarray                # [R] fp32, sigma_next - sigma_cur of this step (negative)
    shell: Dict[str, np.ndarray]
    weights: List[Dict[str, np.ndarray]]

    @property
    def token_lens(self) -> List[int]:
        return [r.n_tokens for r in self.requests]


def make_step_inputs(dims: ModelDims, n_blocks: int, reqs: Sequence[Tuple[int, int, int]], seed: int = 0,
                     n_steps: int = 50) -> StepInputs:
    """Draw order: per request (step index, latent, text tokens, pooled), shell tensors, block tensors.

    Each request sits at its own position of an n_steps-long schedule with sigma = 1 - i/n_steps
    and t = 1000 sigma, as requests of a serving batch are at different steps of their schedules.
    """
    rng = np.random.default_rng(seed)
    requests, latents, texts, pooled, dsig = [], [], [], [], []
    for (hh, ww, n_text) in reqs:
        i = int(rng.integers(0, n_steps))
        sigma, sigma_next = 1.0 - i / n_steps, 1.0 - (i + 1) / n_steps
        requests.append(Request(hh, ww, n_text, 1000.0 * sigma, i))
        latents.append(rng.standard_normal(size=(LATENT_CHANNELS, hh // VAE_FACTOR, ww // VAE_FACTOR), dtype=np.float32))
        texts.append(_normal_bf16(rng, (n_text, dims.hidden), 1.0))
        pooled.append(rng.standard_normal(size=dims.cond_dim, dtype=np.float32))
        dsig.append(np.float32(sigma_next - sigma))
    shell = draw_shell_weights(rng, dims)
    weights = [draw_block_weights(rng, dims) for _ in range(n_blocks)]
    return StepInputs(dims, requests, latents, texts, np.stack(pooled), np.asarray(dsig, dtype=np.float32), shell, weights)
