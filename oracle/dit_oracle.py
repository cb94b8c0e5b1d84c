"""CPU oracle for one DiT denoising step (TEST INFRASTRUCTURE, not a product path).

A plain, slow NumPy fp64 statement of what the GPU library computes: a stack
of adaLN-Zero DiT blocks applied to each request of a packed batch on its own.
Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares no code with the CUDA path and imports neither it nor
torch.

What the paper fixes (Section 2 background and Section 2.1): a denoising step
runs the transformer over a request's *full* latent token set, with attention
giving every token global context; inference is stateless (Section 1); a
request of H x W pixels has (H*W)/16^2 image tokens (Table 1, Section 6.1).
The paper does not spell out the block, so the block below is the standard
adaLN-Zero DiT block with the following readings (each is also listed in the
design notes of the repository):

  * sequential pre-LN block: attention branch, then MLP branch;
  * cond -> modulation is Linear(SiLU(cond)) with bias, split into
    (shift_a, scale_a, gate_a, shift_m, scale_m, gate_m), H each;
  * LayerNorm over the H channels, biased variance, eps inside the root,
    no learned affine;  modulate = LN(x) * (1 + scale) + shift;
  * one weight set for image and text tokens; softmax scale 1/sqrt(d);
    no mask inside a request, no other request visible; no positional term
    unless asked for (below);
  * GELU in its tanh form.

Optional parts, off by default, for the model variants the paper serves (its
FLUX / SD3 class models): per-head RMS-norm of queries and keys with a learned
[d] scale, and a 2-D rotary position term on queries and keys (first d/8
channels of a head unrotated, then a patch-row group and a patch-column group
of equal size, adjacent channel pairs, base 10000; text tokens at (0, 0)).

A second block form, `parallel_block_forward`: one modulation triple, attention
and MLP both read the same modulated LayerNorm output, one output projection
over their concatenation (the "single-stream" blocks of the FLUX family).
A third, `dual_block_forward`: image and text tokens of a request each have
their own block tensors and meet only in attention (the "double-stream" /
MMDiT blocks of the FLUX and SD3 families).

Every function works on fp64 arrays.  Nothing is tiled, fused or reordered
beyond taking query rows in slabs to bound memory (each softmax row is still
the full definition over all keys of the request).

Parity pins (tests/test_oracle_pins.py): hand-derived 2-token cases, softmax
rows summing to one, zero gate => identity, row-permutation equivariance,
packed (explicit block-diagonal mask) == each request alone, closed forms for
LayerNorm / SiLU / GELU / modulation, Table 1 token counts for the packer;
RMS-norm and rotary hand cases, norm preservation and the relative-position
property of the rotary term.
"""
from __future__ import annotations

import math
from typing import Dict, List, Sequence, Tuple

import numpy as np

PATCH_PIXELS = 16

Weights = Dict[str, np.ndarray]


# --------------------------------------------------------------------------
# request packing (integer, exact)
# --------------------------------------------------------------------------
def image_tokens(height: int, width: int) -> int:
    """L = H*W / 16^2 (Section 6.1; Table 1 lists 256/1024/4096/16384)."""
    if height <= 0 or width <= 0 or height % PATCH_PIXELS or width % PATCH_PIXELS:
        raise ValueError("height and width must be positive multiples of 16")
    return (height // PATCH_PIXELS) * (width // PATCH_PIXELS)


def pack_requests(reqs: Sequence[Tuple[int, int, int]]):
    """reqs: (height, width, n_text).  Returns token_lens, cu_seqlens, row_req, row_local.

    Requests keep their input order; rows of request r occupy
    [cu_seqlens[r], cu_seqlens[r+1]); inside a request image tokens come first.
    """
    lens = []
    for (h, w, n_text) in reqs:
        if n_text < 0:
            raise ValueError("negative text token count")
        lens.append(image_tokens(h, w) + n_text)
    cu = [0]
    for l in lens:
        cu.append(cu[-1] + l)
    row_req, row_local = [], []
    for r, l in enumerate(lens):
        for i in range(l):
            row_req.append(r)
            row_local.append(i)
    return (np.array(lens, dtype=np.int32), np.array(cu, dtype=np.int32),
            np.array(row_req, dtype=np.int32), np.array(row_local, dtype=np.int32))


# --------------------------------------------------------------------------
# block pieces
# --------------------------------------------------------------------------
def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def gelu_tanh(z: np.ndarray) -> np.ndarray:
    return 0.5 * z * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)))


def layer_norm(x: np.ndarray, eps: float) -> np.ndarray:
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps)


def adaln_modulation(cond: np.ndarray, w_ada: np.ndarray, b_ada: np.ndarray):
    """cond [C] -> six vectors of H: shift_a, scale_a, gate_a, shift_m, scale_m, gate_m."""
    m = silu(cond) @ w_ada + b_ada
    return tuple(np.split(m, 6))


def modulate(xhat: np.ndarray, shift: np.ndarray, scale: np.ndarray) -> np.ndarray:
    return xhat * (1.0 + scale) + shift


def softmax_rows(s: np.ndarray) -> np.ndarray:
    e = np.exp(s - s.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, n_heads: int,
              rows: np.ndarray | None = None, slab: int = 2048) -> np.ndarray:
    """Multi-head softmax attention over ONE request.  q,k,v: [L, H]; returns [len(rows), H].

    Head j owns columns j*d .. (j+1)*d-1.  `rows` selects query rows (default all).
    """
    L, H = k.shape
    d = H // n_heads
    if rows is not None:
        q = q[rows]
    out = np.empty((q.shape[0], H), dtype=np.float64)
    for j in range(n_heads):
        cols = slice(j * d, (j + 1) * d)
        kj, vj = k[:, cols], v[:, cols]
        for r0 in range(0, q.shape[0], slab):
            s = (q[r0:r0 + slab, cols] @ kj.T) / math.sqrt(d)
            out[r0:r0 + slab, cols] = softmax_rows(s) @ vj
    return out


E4M3_MAX = 448.0


def quantize_e4m3(x: np.ndarray) -> np.ndarray:
    """Nearest value of the 8-bit float with 4 exponent and 3 mantissa bits (bias 7, no infinities,
    largest finite value 448), ties to the even mantissa, larger magnitudes clamped to 448."""
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    _, e = np.frexp(a)                                  # a = m * 2^e, m in [0.5, 1)
    step = np.exp2(np.maximum(e - 1, -6) - 3.0)         # spacing: 2^(exponent - 3), exponent >= -6 (subnormals)
    q = np.minimum(np.rint(a / step) * step, E4M3_MAX)  # rint rounds halves to even
    return np.sign(x) * q


def fp8_linear(h: np.ndarray, w: np.ndarray, b: np.ndarray) -> np.ndarray:
    """h W + b with both operands reduced to e4m3: each row of h is scaled so that its largest
    magnitude maps to 448, each column of W likewise; the product of the quantised operands is
    exact and is scaled back."""
    sa = np.abs(h).max(axis=1, keepdims=True) / E4M3_MAX
    sw = np.abs(w).max(axis=0, keepdims=True) / E4M3_MAX
    sa[sa == 0.0] = 1.0
    sw[sw == 0.0] = 1.0
    return (quantize_e4m3(h / sa) @ quantize_e4m3(w / sw)) * sa * sw + b


def rms_norm_heads(z: np.ndarray, g: np.ndarray, n_heads: int, eps: float) -> np.ndarray:
    """RMS-norm of every head of every row: z_head / sqrt(mean(z_head^2) + eps) * g, g [d]."""
    L, H = z.shape
    zh = z.reshape(L, n_heads, H // n_heads)
    ms = (zh ** 2).mean(axis=-1, keepdims=True)
    return (zh / np.sqrt(ms + eps) * g).reshape(L, H)


def rope_groups(d: int) -> Tuple[int, int]:
    """(d_t, d_axis): the first d/8 channels of a head are not rotated (an index axis that stays at
    position 0); the rest splits evenly into a patch-row group and a patch-column group."""
    d_t = d // 8
    return d_t, (d - d_t) // 2


def rope_2d(z: np.ndarray, positions: np.ndarray, n_heads: int) -> np.ndarray:
    """Rotary position term on every head.  positions [L, 2] = (patch row, patch column); text
    tokens carry (0, 0).  In a group of n channels pair i = channels (2i, 2i+1) of the group turns by
    the angle p * 10000^(-2i/n), p being the row for the first group and the column for the second."""
    L, H = z.shape
    d = H // n_heads
    d_t, n = rope_groups(d)
    out = z.reshape(L, n_heads, d).copy()
    theta = 10000.0 ** (-2.0 * np.arange(n // 2, dtype=np.float64) / n)
    for axis in range(2):
        ang = positions[:, axis].astype(np.float64)[:, None] * theta[None, :]        # [L, n/2]
        c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
        lo = d_t + axis * n
        a, b = out[:, :, lo:lo + n:2].copy(), out[:, :, lo + 1:lo + n:2].copy()
        out[:, :, lo:lo + n:2] = a * c - b * s
        out[:, :, lo + 1:lo + n:2] = a * s + b * c
    return out.reshape(L, H)


def patch_positions(height: int, width: int, n_text: int) -> np.ndarray:
    """[L, 2] (patch row, patch column) of a request's tokens: image tokens row-major, text at (0, 0)."""
    gh, gw = height // PATCH_PIXELS, width // PATCH_PIXELS
    py, px = np.meshgrid(np.arange(gh), np.arange(gw), indexing="ij")
    img = np.stack([py.reshape(-1), px.reshape(-1)], axis=1)
    return np.concatenate([img, np.zeros((n_text, 2), dtype=img.dtype)], axis=0)


def block_forward(x: np.ndarray, cond: np.ndarray, w: Weights, n_heads: int, eps: float,
                  rows: np.ndarray | None = None, taps: dict | None = None,
                  positions: np.ndarray | None = None, fp8: bool = False) -> np.ndarray:
    """One adaLN-Zero DiT block on one request.  x [L, H], cond [C] -> [L, H].

    With `rows`, only those output rows are produced (keys and values still
    come from every row of the request); used to sample outputs of long
    sequences.  `taps`, if given, receives the intermediates h1, qkv, a, x_mid,
    h2, u for per-kernel comparisons.

    Two optional parts of the model variants: if `w` holds "q_norm" / "k_norm"
    ([d] each), queries and keys are RMS-normed per head (same eps) before
    attention; if `positions` [L, 2] is given, queries and keys then get the
    2-D rotary term.  The taps' qkv is taken after both.

    With `fp8`, the two products that read a LayerNorm output (QKV and the MLP up-projection) take
    their operands through fp8_linear; everything else is unchanged.
    """
    H = x.shape[1]
    lin = fp8_linear if fp8 else (lambda a, ww, bb: a @ ww + bb)
    shift_a, scale_a, gate_a, shift_m, scale_m, gate_m = adaln_modulation(cond, w["w_ada"], w["b_ada"])
    h = modulate(layer_norm(x, eps), shift_a, scale_a)
    qkv = lin(h, w["w_qkv"], w["b_qkv"])
    q, k, v = qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:]
    if "q_norm" in w:
        q = rms_norm_heads(q, w["q_norm"], n_heads, eps)
        k = rms_norm_heads(k, w["k_norm"], n_heads, eps)
    if positions is not None:
        q, k = rope_2d(q, positions, n_heads), rope_2d(k, positions, n_heads)
    if "q_norm" in w or positions is not None:
        qkv = np.concatenate([q, k, v], axis=1)
    a = attention(q, k, v, n_heads, rows)
    xr = x if rows is None else x[rows]
    x_mid = xr + gate_a * (a @ w["w_o"] + w["b_o"])
    h2 = modulate(layer_norm(x_mid, eps), shift_m, scale_m)
    u = gelu_tanh(lin(h2, w["w_fc1"], w["b_fc1"]))
    y = x_mid + gate_m * (u @ w["w_fc2"] + w["b_fc2"])
    if taps is not None:
        taps.update(h1=h, qkv=qkv, a=a, x_mid=x_mid, h2=h2, u=u)
    return y


def parallel_block_forward(x: np.ndarray, cond: np.ndarray, w: Weights, n_heads: int, eps: float,
                           rows: np.ndarray | None = None, taps: dict | None = None,
                           positions: np.ndarray | None = None, fp8: bool = False) -> np.ndarray:
    """The parallel (single-modulation) form of the block: attention and the MLP read the same
    modulated LayerNorm output, their results are concatenated and share one output projection:

        (shift, scale, gate) = SiLU(cond) W_ada + b_ada                    W_ada [C, 3H]
        h = LN(x) (1 + scale) + shift
        a = attention(h W_qkv + b_qkv),   u = gelu_tanh(h W_fc1 + b_fc1)
        y = x + gate * ([a | u] W_out + b_out)                             W_out [H + F, H]

    Optional q_norm / k_norm and `positions` act on queries and keys as in block_forward.
    """
    H = x.shape[1]
    lin = fp8_linear if fp8 else (lambda a, ww, bb: a @ ww + bb)
    shift, scale, gate = np.split(silu(cond) @ w["w_ada"] + w["b_ada"], 3)
    h = modulate(layer_norm(x, eps), shift, scale)
    qkv = lin(h, w["w_qkv"], w["b_qkv"])
    q, k, v = qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:]
    if "q_norm" in w:
        q = rms_norm_heads(q, w["q_norm"], n_heads, eps)
        k = rms_norm_heads(k, w["k_norm"], n_heads, eps)
    if positions is not None:
        q, k = rope_2d(q, positions, n_heads), rope_2d(k, positions, n_heads)
    a = attention(q, k, v, n_heads, rows)
    hr, xr = (h, x) if rows is None else (h[rows], x[rows])
    u = gelu_tanh(lin(hr, w["w_fc1"], w["b_fc1"]))
    y = xr + gate * (np.concatenate([a, u], axis=1) @ w["w_out"] + w["b_out"])
    if taps is not None:
        taps.update(h1=h, qkv=np.concatenate([q, k, v], axis=1), a=a, u=u)
    return y


def dual_block_forward(x: np.ndarray, cond: np.ndarray, w: Weights, n_img: int, n_heads: int, eps: float,
                       rows: np.ndarray | None = None, taps: dict | None = None,
                       positions: np.ndarray | None = None) -> np.ndarray:
    """The two-stream form of the block: the first n_img rows (image tokens) use the tensors of
    `w`, the remaining rows (text tokens) use those of w["txt"]; each stream has its own
    modulation, projections, MLP and (optionally) q/k norm scales.  Only attention mixes them: it
    runs once over all rows of the request, queries, keys and values taken stream by stream.
    """
    L, H = x.shape
    streams = [(slice(0, n_img), w), (slice(n_img, L), w["txt"])]
    mods, qs, ks, vs, hs = [], [], [], [], []
    for sl, ws in streams:
        m = adaln_modulation(cond, ws["w_ada"], ws["b_ada"])
        h = modulate(layer_norm(x[sl], eps), m[0], m[1])
        qkv = h @ ws["w_qkv"] + ws["b_qkv"]
        q, k, v = qkv[:, :H], qkv[:, H:2 * H], qkv[:, 2 * H:]
        if "q_norm" in ws:
            q = rms_norm_heads(q, ws["q_norm"], n_heads, eps)
            k = rms_norm_heads(k, ws["k_norm"], n_heads, eps)
        mods.append(m); hs.append(h); qs.append(q); ks.append(k); vs.append(v)
    q, k, v = np.concatenate(qs), np.concatenate(ks), np.concatenate(vs)
    if positions is not None:
        q, k = rope_2d(q, positions, n_heads), rope_2d(k, positions, n_heads)
    a = attention(q, k, v, n_heads)                      # all rows: both streams need their own
    y = np.empty_like(x)
    u_all = []
    for (sl, ws), m in zip(streams, mods):
        x_mid = x[sl] + m[2] * (a[sl] @ ws["w_o"] + ws["b_o"])
        h2 = modulate(layer_norm(x_mid, eps), m[3], m[4])
        u = gelu_tanh(h2 @ ws["w_fc1"] + ws["b_fc1"])
        y[sl] = x_mid + m[5] * (u @ ws["w_fc2"] + ws["b_fc2"])
        u_all.append(u)
    if taps is not None:
        taps.update(h1=np.concatenate(hs), qkv=np.concatenate([q, k, v], axis=1), a=a, u=np.concatenate(u_all))
    return y if rows is None else y[rows]


def any_block_forward(x, cond, w: Weights, n_heads: int, eps: float, n_img: int | None = None, **kw) -> np.ndarray:
    """Dispatch on the block's form: a two-stream block holds "txt" (the text stream's tensors), a
    parallel block holds "w_out".  n_img (image rows of the request) is needed by two-stream blocks."""
    if "txt" in w:
        return dual_block_forward(x, cond, w, n_img, n_heads, eps, **kw)
    return (parallel_block_forward if "w_out" in w else block_forward)(x, cond, w, n_heads, eps, **kw)


def stack_forward_alone(x: np.ndarray, cond: np.ndarray, blocks: Sequence[Weights],
                        n_heads: int, eps: float, positions: np.ndarray | None = None,
                        n_img: int | None = None, fp8: bool = False) -> np.ndarray:
    """A stack of blocks on one request run by itself (fp8: sequential and parallel forms only)."""
    for w in blocks:
        kw = {"fp8": True} if fp8 else {}
        x = any_block_forward(x, cond, w, n_heads, eps, n_img=n_img, positions=positions, **kw)
    return x


def step_forward(packed: np.ndarray, token_lens: Sequence[int], cond: np.ndarray,
                 blocks: Sequence[Weights], n_heads: int, eps: float,
                 positions: Sequence[np.ndarray] | None = None,
                 n_imgs: Sequence[int] | None = None, fp8: bool = False) -> np.ndarray:
    """One denoising step over a packed batch: each request through the stack on its own."""
    out = np.empty_like(packed)
    p = 0
    for r, l in enumerate(token_lens):
        out[p:p + l] = stack_forward_alone(packed[p:p + l], cond[r], blocks, n_heads, eps,
                                           None if positions is None else positions[r],
                                           None if n_imgs is None else n_imgs[r], fp8)
        p += l
    return out


def step_forward_masked(packed: np.ndarray, token_lens: Sequence[int], cond: np.ndarray,
                        blocks: Sequence[Weights], n_heads: int, eps: float) -> np.ndarray:
    """Second, independent statement of the packed step (small cases only).

    Works on the whole [T, H] batch at once: per-row modulation vectors looked
    up through row -> request, and ONE T x T score matrix per head with an
    explicit block-diagonal mask (-inf outside a row's own request).
    """
    T, H = packed.shape
    d = H // n_heads
    row_req = np.repeat(np.arange(len(token_lens)), token_lens)
    same = row_req[:, None] == row_req[None, :]
    x = packed.copy()
    for w in blocks:
        mod = np.stack([silu(c) @ w["w_ada"] + w["b_ada"] for c in cond])[row_req]   # [T, 6H]
        sh_a, sc_a, g_a, sh_m, sc_m, g_m = (mod[:, i * H:(i + 1) * H] for i in range(6))
        h = layer_norm(x, eps) * (1.0 + sc_a) + sh_a
        qkv = h @ w["w_qkv"] + w["b_qkv"]
        a = np.empty_like(x)
        for j in range(n_heads):
            q = qkv[:, j * d:(j + 1) * d]
            k = qkv[:, H + j * d:H + (j + 1) * d]
            v = qkv[:, 2 * H + j * d:2 * H + (j + 1) * d]
            s = np.where(same, (q @ k.T) / math.sqrt(d), -np.inf)
            a[:, j * d:(j + 1) * d] = softmax_rows(s) @ v
        x = x + g_a * (a @ w["w_o"] + w["b_o"])
        h = layer_norm(x, eps) * (1.0 + sc_m) + sh_m
        x = x + g_m * (gelu_tanh(h @ w["w_fc1"] + w["b_fc1"]) @ w["w_fc2"] + w["b_fc2"])
    return x


def block_forward_scalar(x: Sequence[Sequence[float]], cond: Sequence[float], w: Weights,
                         n_heads: int, eps: float) -> List[List[float]]:
    """Third statement, pure-Python scalar loops (tiny cases only): no NumPy arithmetic."""
    L, H = len(x), len(x[0])
    C = len(cond)
    d = H // n_heads
    W = {k: np.asarray(v).tolist() for k, v in w.items()}
    sc = [c / (1.0 + math.exp(-c)) for c in cond]
    m = [sum(sc[i] * W["w_ada"][i][o] for i in range(C)) + W["b_ada"][o] for o in range(6 * H)]
    part = [m[i * H:(i + 1) * H] for i in range(6)]

    def ln_mod(row, shift, scale):
        mu = sum(row) / H
        var = sum((t - mu) ** 2 for t in row) / H
        return [(row[c] - mu) / math.sqrt(var + eps) * (1.0 + scale[c]) + shift[c] for c in range(H)]

    def linear(row, wname, bname):
        wm, b = W[wname], W[bname]
        return [sum(row[i] * wm[i][o] for i in range(len(row))) + b[o] for o in range(len(b))]

    h = [ln_mod(r, part[0], part[1]) for r in x]
    qkv = [linear(r, "w_qkv", "b_qkv") for r in h]
    a = [[0.0] * H for _ in range(L)]
    for j in range(n_heads):
        for i in range(L):
            s = [sum(qkv[i][j * d + c] * qkv[t][H + j * d + c] for c in range(d)) / math.sqrt(d) for t in range(L)]
            e = [math.exp(v) for v in s]
            z = sum(e)
            for c in range(d):
                a[i][j * d + c] = sum(e[t] / z * qkv[t][2 * H + j * d + c] for t in range(L))
    proj = [linear(r, "w_o", "b_o") for r in a]
    xm = [[x[i][c] + part[2][c] * proj[i][c] for c in range(H)] for i in range(L)]
    h2 = [ln_mod(r, part[3], part[4]) for r in xm]
    pre = [linear(r, "w_fc1", "b_fc1") for r in h2]
    u = [[0.5 * z * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z * z * z))) for z in r] for r in pre]
    f2 = [linear(r, "w_fc2", "b_fc2") for r in u]
    return [[xm[i][c] + part[5][c] * f2[i][c] for c in range(H)] for i in range(L)]


def error_metric(got: np.ndarray, ref: np.ndarray) -> float:
    """max|got - ref| / rms(ref) over one request's outputs."""
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.abs(np.asarray(got, dtype=np.float64) - ref).max() / math.sqrt(np.mean(ref ** 2)))
