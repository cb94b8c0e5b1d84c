"""Pins for the optional model-variant parts of the block oracle: per-head RMS-norm of queries and
keys, and the 2-D rotary position term."""
import math

import numpy as np
import pytest

from oracle import dit_oracle as O


def test_rms_norm_hand_cases():
    # one head of 4: [3, 4, 0, 0] has mean square 25/4, so the normed vector is [1.2, 1.6, 0, 0]
    z = np.array([[3.0, 4.0, 0.0, 0.0]])
    assert np.allclose(O.rms_norm_heads(z, np.ones(4), 1, 0.0), [[1.2, 1.6, 0.0, 0.0]], atol=1e-15)
    # the learned scale multiplies channel by channel
    assert np.allclose(O.rms_norm_heads(z, np.array([2.0, -1.0, 5.0, 7.0]), 1, 0.0), [[2.4, -1.6, 0.0, 0.0]], atol=1e-15)
    # two heads are normed separately: a constant head c becomes sign(c)
    z = np.array([[5.0, 5.0, -0.01, -0.01]])
    assert np.allclose(O.rms_norm_heads(z, np.ones(2), 2, 0.0), [[1.0, 1.0, -1.0, -1.0]], atol=1e-15)
    # eps sits inside the root: a zero head stays zero, a head of 1s becomes 1/sqrt(1 + eps)
    z = np.array([[0.0, 0.0, 1.0, 1.0]])
    got = O.rms_norm_heads(z, np.ones(2), 2, 0.21)
    assert np.allclose(got, [[0.0, 0.0, 1 / 1.1, 1 / 1.1]], atol=1e-15)
    # scale invariance and unit mean square (eps = 0)
    rng = np.random.default_rng(0)
    z = rng.standard_normal((7, 96))
    a = O.rms_norm_heads(z, np.ones(32), 3, 0.0)
    assert np.allclose(a, O.rms_norm_heads(17.0 * z, np.ones(32), 3, 0.0), atol=1e-14)
    assert np.allclose((a.reshape(7, 3, 32) ** 2).mean(-1), 1.0, atol=1e-14)


def test_rope_groups_for_the_two_head_sizes():
    assert O.rope_groups(128) == (16, 56)
    assert O.rope_groups(64) == (8, 28)
    assert O.rope_groups(32) == (4, 14)


def test_rope_hand_case():
    # one head of 32: channels 0..3 fixed, 4..17 turn with the row, 18..31 with the column.
    z = np.zeros((1, 32))
    z[0, 2] = 9.0             # unrotated group
    z[0, 4], z[0, 5] = 1.0, 0.0       # row group, pair 0: frequency 1
    z[0, 16], z[0, 17] = 0.0, 2.0     # row group, pair 6: frequency 10000^(-12/14)
    z[0, 18], z[0, 19] = 3.0, 4.0     # column group, pair 0: frequency 1
    py, px = 2, 5
    out = O.rope_2d(z, np.array([[py, px]]), 1)[0]
    assert out[2] == 9.0
    assert out[4] == pytest.approx(math.cos(2.0), abs=1e-15) and out[5] == pytest.approx(math.sin(2.0), abs=1e-15)
    a = py * 10000.0 ** (-12.0 / 14.0)
    assert out[16] == pytest.approx(-2.0 * math.sin(a), abs=1e-15) and out[17] == pytest.approx(2.0 * math.cos(a), abs=1e-15)
    assert out[18] == pytest.approx(3 * math.cos(5.0) - 4 * math.sin(5.0), abs=1e-14)
    assert out[19] == pytest.approx(3 * math.sin(5.0) + 4 * math.cos(5.0), abs=1e-14)
    untouched = [i for i in range(32) if i not in (2, 4, 5, 16, 17, 18, 19)]
    assert np.array_equal(out[untouched], np.zeros(len(untouched)))


def test_rope_is_a_rotation_and_encodes_relative_position():
    rng = np.random.default_rng(1)
    heads, d = 3, 64
    q, k = rng.standard_normal((1, heads * d)), rng.standard_normal((1, heads * d))
    # position (0, 0) (text tokens) leaves the vector as it is
    assert np.array_equal(O.rope_2d(q, np.array([[0, 0]]), heads), q)
    # per-head norms survive any position
    r = O.rope_2d(q, np.array([[37, 120]]), heads)
    assert np.allclose((r.reshape(heads, d) ** 2).sum(-1), (q.reshape(heads, d) ** 2).sum(-1), rtol=1e-13)
    # the score of a query at p and a key at p' depends on p - p' only, head by head
    def scores(pq, pk):
        a = O.rope_2d(q, np.array([pq]), heads).reshape(heads, d)
        b = O.rope_2d(k, np.array([pk]), heads).reshape(heads, d)
        return (a * b).sum(-1)
    base = scores((10, 3), (4, 9))
    assert np.allclose(scores((10 + 50, 3 + 20), (4 + 50, 9 + 20)), base, atol=1e-12)
    assert not np.allclose(scores((10, 3), (5, 9)), base, atol=1e-3)
    # rows and columns act on different channels: moving only the column leaves the row group's part alone
    a = O.rope_2d(q, np.array([[6, 1]]), heads).reshape(heads, d)
    b = O.rope_2d(q, np.array([[6, 77]]), heads).reshape(heads, d)
    assert np.array_equal(a[:, :8 + 28], b[:, :8 + 28]) and not np.allclose(a[:, 8 + 28:], b[:, 8 + 28:])


def test_patch_positions():
    p = O.patch_positions(32, 48, 2)            # 2 x 3 patches, then two text tokens
    assert p.tolist() == [[0, 0], [0, 1], [0, 2], [1, 0], [1, 1], [1, 2], [0, 0], [0, 0]]


def _block(rng, H, F, C, d=None):
    w = {"w_ada": rng.standard_normal((C, 6 * H)) * 0.1, "b_ada": rng.standard_normal(6 * H) * 0.1,
         "w_qkv": rng.standard_normal((H, 3 * H)) * 0.2, "b_qkv": rng.standard_normal(3 * H) * 0.1,
         "w_o": rng.standard_normal((H, H)) * 0.2, "b_o": np.zeros(H),
         "w_fc1": rng.standard_normal((H, F)) * 0.2, "b_fc1": np.zeros(F),
         "w_fc2": rng.standard_normal((F, H)) * 0.2, "b_fc2": np.zeros(H)}
    if d:
        w["q_norm"] = 1.0 + 0.1 * rng.standard_normal(d)
        w["k_norm"] = 1.0 + 0.1 * rng.standard_normal(d)
    return w


def test_block_with_variants_reduces_to_the_plain_block():
    rng = np.random.default_rng(2)
    H, heads, L = 64, 2, 6
    w = _block(rng, H, 128, 8)
    x, cond = rng.standard_normal((L, H)), rng.standard_normal(8)
    plain = O.block_forward(x, cond, w, heads, 1e-6)
    # all tokens at position (0, 0): the rotary term is the identity
    assert np.array_equal(O.block_forward(x, cond, w, heads, 1e-6, positions=np.zeros((L, 2), dtype=int)), plain)
    # a common shift of all positions changes no score, hence nothing
    pos = np.array([[0, 0], [0, 1], [1, 0], [1, 1], [2, 0], [2, 1]])
    a = O.block_forward(x, cond, w, heads, 1e-6, positions=pos)
    b = O.block_forward(x, cond, w, heads, 1e-6, positions=pos + np.array([7, 30]))
    assert np.allclose(a, b, atol=1e-11) and not np.allclose(a, plain, atol=1e-3)
    # RMS-norm of q and k makes the block blind to the scale of W_q and W_k (eps = 0, zero q/k bias)
    wn = dict(_block(rng, H, 128, 8, d=32))
    wn["b_qkv"] = np.concatenate([np.zeros(2 * H), wn["b_qkv"][2 * H:]])
    ref = O.block_forward(x, cond, wn, heads, 0.0, positions=pos)
    ws = dict(wn)
    ws["w_qkv"] = np.concatenate([3.0 * wn["w_qkv"][:, :H], 0.25 * wn["w_qkv"][:, H:2 * H], wn["w_qkv"][:, 2 * H:]], axis=1)
    # eps = 0 also in LayerNorm here; harmless for random rows
    assert np.allclose(O.block_forward(x, cond, ws, heads, 0.0, positions=pos), ref, atol=1e-11)


def test_taps_hold_normed_and_rotated_queries():
    rng = np.random.default_rng(3)
    H, heads, L = 64, 2, 4
    w = _block(rng, H, 128, 8, d=32)
    x, cond = rng.standard_normal((L, H)), rng.standard_normal(8)
    pos = np.array([[0, 0], [0, 1], [1, 0], [1, 1]])
    taps = {}
    O.block_forward(x, cond, w, heads, 1e-6, taps=taps, positions=pos)
    raw = taps["h1"] @ w["w_qkv"] + w["b_qkv"]
    want_q = O.rope_2d(O.rms_norm_heads(raw[:, :H], w["q_norm"], heads, 1e-6), pos, heads)
    assert np.array_equal(taps["qkv"][:, :H], want_q)
    assert np.array_equal(taps["qkv"][:, 2 * H:], raw[:, 2 * H:])      # values are neither normed nor rotated


# ----------------------------------------------------------------------------- the parallel block form
def test_parallel_block_reduces_to_halves_of_the_sequential_block():
    rng = np.random.default_rng(7)
    H, F, C, heads, L = 64, 128, 8, 2, 5
    w = _block(rng, H, F, C)
    w["b_o"] = rng.standard_normal(H) * 0.1
    w["b_fc2"] = rng.standard_normal(H) * 0.1
    x, cond = rng.standard_normal((L, H)), rng.standard_normal(C)
    sh_a, sc_a, g_a, sh_m, sc_m, g_m = np.split(w["w_ada"], 6, axis=1)
    bsh_a, bsc_a, bg_a, bsh_m, bsc_m, bg_m = np.split(w["b_ada"], 6)
    zero_w, zero_b = np.zeros_like(g_a), np.zeros_like(bg_a)

    # (1) attention half: the parallel block whose output projection ignores the MLP columns equals the
    #     sequential block with a zero MLP gate
    par = {"w_ada": np.concatenate([sh_a, sc_a, g_a], axis=1), "b_ada": np.concatenate([bsh_a, bsc_a, bg_a]),
           "w_qkv": w["w_qkv"], "b_qkv": w["b_qkv"], "w_fc1": w["w_fc1"], "b_fc1": w["b_fc1"],
           "w_out": np.concatenate([w["w_o"], np.zeros((F, H))], axis=0), "b_out": w["b_o"]}
    seq = dict(w, w_ada=np.concatenate([sh_a, sc_a, g_a, sh_m, sc_m, zero_w], axis=1),
               b_ada=np.concatenate([bsh_a, bsc_a, bg_a, bsh_m, bsc_m, zero_b]))
    assert np.allclose(O.parallel_block_forward(x, cond, par, heads, 1e-6), O.block_forward(x, cond, seq, heads, 1e-6), atol=1e-13)

    # (2) MLP half: ignoring the attention columns equals the sequential block with a zero attention
    #     gate, whose second LayerNorm then sees x itself
    par2 = dict(par, w_ada=np.concatenate([sh_m, sc_m, g_m], axis=1), b_ada=np.concatenate([bsh_m, bsc_m, bg_m]),
                w_out=np.concatenate([np.zeros((H, H)), w["w_fc2"]], axis=0), b_out=w["b_fc2"])
    seq2 = dict(w, w_ada=np.concatenate([sh_a, sc_a, zero_w, sh_m, sc_m, g_m], axis=1),
                b_ada=np.concatenate([bsh_a, bsc_a, zero_b, bsh_m, bsc_m, bg_m]))
    assert np.allclose(O.parallel_block_forward(x, cond, par2, heads, 1e-6), O.block_forward(x, cond, seq2, heads, 1e-6), atol=1e-13)

    # (3) the two halves add up: with one modulation triple, full = x + (attention half - x) + (MLP half - x)
    tri_w, tri_b = np.concatenate([sh_a, sc_a, g_a], axis=1), np.concatenate([bsh_a, bsc_a, bg_a])
    full = dict(par, w_ada=tri_w, b_ada=tri_b, w_out=np.concatenate([w["w_o"], w["w_fc2"]], axis=0), b_out=w["b_o"] + w["b_fc2"])
    half_a = dict(full, w_out=np.concatenate([w["w_o"], np.zeros((F, H))], axis=0), b_out=w["b_o"])
    half_m = dict(full, w_out=np.concatenate([np.zeros((H, H)), w["w_fc2"]], axis=0), b_out=w["b_fc2"])
    ya, ym = (O.parallel_block_forward(x, cond, ww, heads, 1e-6) for ww in (half_a, half_m))
    assert np.allclose(O.parallel_block_forward(x, cond, full, heads, 1e-6), ya + ym - x, atol=1e-13)


def test_parallel_block_zero_gate_rows_and_dispatch():
    rng = np.random.default_rng(8)
    H, F, C, heads, L = 64, 128, 8, 2, 6
    par = {"w_ada": rng.standard_normal((C, 3 * H)) * 0.1, "b_ada": rng.standard_normal(3 * H) * 0.1,
           "w_qkv": rng.standard_normal((H, 3 * H)) * 0.2, "b_qkv": rng.standard_normal(3 * H) * 0.1,
           "w_fc1": rng.standard_normal((H, F)) * 0.2, "b_fc1": rng.standard_normal(F) * 0.1,
           "w_out": rng.standard_normal((H + F, H)) * 0.2, "b_out": rng.standard_normal(H) * 0.1}
    x, cond = rng.standard_normal((L, H)), rng.standard_normal(C)
    y = O.parallel_block_forward(x, cond, par, heads, 1e-6)
    # zero gate: identity
    z = dict(par, w_ada=par["w_ada"].copy(), b_ada=par["b_ada"].copy())
    z["w_ada"][:, 2 * H:] = 0.0
    z["b_ada"][2 * H:] = 0.0
    assert np.array_equal(O.parallel_block_forward(x, cond, z, heads, 1e-6), x)
    # row subset == the same rows of the full result
    rows = np.array([4, 1])
    assert np.allclose(O.parallel_block_forward(x, cond, par, heads, 1e-6, rows=rows), y[rows], atol=1e-14)
    # a stack mixes the two forms by what each block holds
    seq = _block(rng, H, F, C)
    want = O.parallel_block_forward(O.block_forward(x, cond, seq, heads, 1e-6), cond, par, heads, 1e-6)
    assert np.array_equal(O.stack_forward_alone(x, cond, [seq, par], heads, 1e-6), want)


# ----------------------------------------------------------------------------- the two-stream block form
def test_dual_block_reduces_to_the_plain_block():
    rng = np.random.default_rng(9)
    H, F, C, heads, L, n_img = 64, 128, 8, 2, 7, 4
    w_img, w_txt = _block(rng, H, F, C, d=32), _block(rng, H, F, C, d=32)
    x, cond = rng.standard_normal((L, H)), rng.standard_normal(C)
    pos = np.array([[0, 0], [0, 1], [1, 0], [1, 1], [0, 0], [0, 0], [0, 0]])
    # same tensors in both streams: the plain block
    same = dict(w_img, txt=w_img)
    assert np.allclose(O.dual_block_forward(x, cond, same, n_img, heads, 1e-6, positions=pos),
                       O.block_forward(x, cond, w_img, heads, 1e-6, positions=pos), atol=1e-13)
    dual = dict(w_img, txt=w_txt)
    # no text rows: the image stream's plain block; no image rows: the text stream's
    assert np.allclose(O.dual_block_forward(x, cond, dual, L, heads, 1e-6), O.block_forward(x, cond, w_img, heads, 1e-6), atol=1e-13)
    assert np.allclose(O.dual_block_forward(x, cond, dual, 0, heads, 1e-6), O.block_forward(x, cond, w_txt, heads, 1e-6), atol=1e-13)
    # different tensors: a different result, and the boundary matters
    y = O.dual_block_forward(x, cond, dual, n_img, heads, 1e-6, positions=pos)
    assert not np.allclose(y, O.block_forward(x, cond, w_img, heads, 1e-6, positions=pos), atol=1e-3)
    assert not np.allclose(y, O.dual_block_forward(x, cond, dual, n_img + 1, heads, 1e-6, positions=pos), atol=1e-3)


def test_dual_block_streams_meet_only_in_attention():
    rng = np.random.default_rng(10)
    H, F, C, heads, L, n_img = 64, 128, 8, 2, 6, 4
    w_img, w_txt = _block(rng, H, F, C), _block(rng, H, F, C)
    x, cond = rng.standard_normal((L, H)), rng.standard_normal(C)
    dual = dict(w_img, txt=w_txt)
    y = O.dual_block_forward(x, cond, dual, n_img, heads, 1e-6)
    # zero gates in the text stream: text rows pass through, image rows still change (and still see
    # the text keys and values, which do not depend on the gates)
    wz = dict(w_txt, w_ada=w_txt["w_ada"].copy(), b_ada=w_txt["b_ada"].copy())
    for g in (2, 5):
        wz["w_ada"][:, g * H:(g + 1) * H] = 0.0
        wz["b_ada"][g * H:(g + 1) * H] = 0.0
    yz = O.dual_block_forward(x, cond, dict(w_img, txt=wz), n_img, heads, 1e-6)
    assert np.array_equal(yz[n_img:], x[n_img:])
    assert np.allclose(yz[:n_img], y[:n_img], atol=1e-13)
    # text values projected to zero: image rows attend to nothing of the text but its softmax mass;
    # hand check on the attention tap: rows of `a` are convex combinations of the value rows
    taps = {}
    O.dual_block_forward(x, cond, dual, n_img, heads, 1e-6, taps=taps)
    v = taps["qkv"][:, 2 * H:]
    a = taps["a"]
    for j in range(heads):
        cols = slice(j * 32, (j + 1) * 32)
        assert (a[:, cols].max(0) <= v[:, cols].max(0) + 1e-12).all() and (a[:, cols].min(0) >= v[:, cols].min(0) - 1e-12).all()
    # the text stream's MLP does not touch image rows: change only w_fc2 of the text stream
    w2 = dict(w_txt, w_fc2=w_txt["w_fc2"] * 3.0)
    y2 = O.dual_block_forward(x, cond, dict(w_img, txt=w2), n_img, heads, 1e-6)
    assert np.array_equal(y2[:n_img], y[:n_img]) and not np.allclose(y2[n_img:], y[n_img:], atol=1e-3)
    # row subset and stack dispatch
    assert np.array_equal(O.dual_block_forward(x, cond, dual, n_img, heads, 1e-6, rows=np.array([5, 0])), y[[5, 0]])
    assert np.array_equal(O.stack_forward_alone(x, cond, [dual], heads, 1e-6, n_img=n_img), y)


# ----------------------------------------------------------------------------- fp8 (e4m3) operands
def test_e4m3_grid():
    q = O.quantize_e4m3
    # representable values stay as they are, both signs
    vals = np.array([0.0, 2.0 ** -9, 2.0 ** -6, 0.875 * 2.0 ** -6, 1.0, 1.125, 1.875, 240.0, 448.0, -3.5, -0.0625])
    assert np.array_equal(q(vals), vals)
    # ties go to the even mantissa; everything beyond 448 is clamped
    assert q(1.0625) == 1.0 and q(1.1875) == 1.25 and q(1.0626) == 1.125
    assert q(2.0 ** -10) == 0.0 and q(3 * 2.0 ** -10) == 2.0 ** -8 and q(2.0 ** -10 * 1.01) == 2.0 ** -9
    assert q(464.0) == 448.0 and q(1e6) == 448.0 and q(-1e6) == -448.0 and q(447.0) == 448.0 and q(431.0) == 416.0
    # the format has 126 positive finite values: 7 subnormals and 15 binades of 8 values, less the NaN code
    grid = np.unique(q(np.linspace(0.0, 500.0, 2_000_001)))
    sub = np.unique(q(np.linspace(0.0, 2.0 ** -6, 100_001)))
    assert len(np.union1d(grid, sub)) - 1 == 126
    # relative error of a normal value is at most 2^-4
    x = np.exp(np.random.default_rng(0).uniform(np.log(2.0 ** -6), np.log(448.0), 10000))
    assert (np.abs(q(x) - x) / x).max() <= 2.0 ** -4


def test_fp8_linear_is_exact_on_grid_operands_and_close_otherwise():
    rng = np.random.default_rng(1)
    # operands already on the e4m3 grid with row / column maxima of 448: nothing is lost
    h = O.quantize_e4m3(rng.uniform(-448, 448, (5, 16))); h[:, 0] = 448.0
    w = O.quantize_e4m3(rng.uniform(-448, 448, (16, 7))); w[0, :] = -448.0
    b = rng.standard_normal(7)
    assert np.allclose(O.fp8_linear(h, w, b), h @ w + b, rtol=1e-14)
    # scaling a row of h or a column of W scales the same row / column of the product exactly
    # (powers of two keep the quantised mantissas)
    h2, w2 = rng.standard_normal((6, 64)), rng.standard_normal((64, 9)) * 0.02
    base = O.fp8_linear(h2, w2, np.zeros(9))
    hs = h2.copy(); hs[2] *= 8.0
    ws = w2.copy(); ws[:, 4] *= 0.25
    assert np.array_equal(O.fp8_linear(hs, w2, np.zeros(9))[2], base[2] * 8.0)
    assert np.array_equal(O.fp8_linear(h2, ws, np.zeros(9))[:, 4], base[:, 4] * 0.25)
    # and the result is a few per cent from the exact product
    exact = h2 @ w2
    assert 1e-3 < O.error_metric(base, exact) < 0.3
    # zero rows and columns do not divide by zero
    hz = h2.copy(); hz[1] = 0.0
    assert np.isfinite(O.fp8_linear(hz, w2, np.zeros(9))).all()


def test_fp8_block_is_the_plain_block_with_two_products_swapped():
    rng = np.random.default_rng(2)
    H, F, C, heads, L = 64, 128, 8, 2, 5
    w = _block(rng, H, F, C)
    x, cond = rng.standard_normal((L, H)), rng.standard_normal(C)
    taps8, taps = {}, {}
    y8 = O.block_forward(x, cond, w, heads, 1e-6, taps=taps8, fp8=True)
    y = O.block_forward(x, cond, w, heads, 1e-6, taps=taps)
    assert np.array_equal(taps8["h1"], taps["h1"])                          # LayerNorm is untouched
    assert np.array_equal(taps8["qkv"], O.fp8_linear(taps["h1"], w["w_qkv"], w["b_qkv"]))
    assert 1e-4 < O.error_metric(y8, y) < 0.2


# ----------------------------------------------------------------------------- e4m3 operands for all four products
def test_fp8_all_products_block_is_the_plain_block_with_four_products_swapped():
    from oracle import fp8_oracle as F8
    rng = np.random.default_rng(3)
    H, F, C, heads, L = 64, 128, 8, 2, 7
    w = _block(rng, H, F, C)
    w["b_o"], w["b_fc2"] = rng.standard_normal(H) * 0.1, rng.standard_normal(H) * 0.1
    x, cond = rng.standard_normal((L, H)), rng.standard_normal(C)
    # quantising no product is the exact block; quantising QKV and the up-projection is dit_oracle's fp8=True
    assert np.array_equal(F8.block_forward_fp8(x, cond, w, heads, 1e-6, quantise=()), O.block_forward(x, cond, w, heads, 1e-6))
    assert np.array_equal(F8.block_forward_fp8(x, cond, w, heads, 1e-6, quantise=("qkv", "fc1")),
                          O.block_forward(x, cond, w, heads, 1e-6, fp8=True))
    # each product of the all-four block is fp8_linear of the tap that feeds it
    t = {}
    y = F8.block_forward_fp8(x, cond, w, heads, 1e-6, taps=t)
    m = O.adaln_modulation(cond, w["w_ada"], w["b_ada"])
    assert np.array_equal(t["qkv"], O.fp8_linear(t["h1"], w["w_qkv"], w["b_qkv"]))
    assert np.array_equal(t["x_mid"], x + m[2] * O.fp8_linear(t["a"], w["w_o"], w["b_o"]))
    assert np.array_equal(t["u"], O.gelu_tanh(O.fp8_linear(t["h2"], w["w_fc1"], w["b_fc1"])))
    assert np.array_equal(y, t["x_mid"] + m[5] * O.fp8_linear(t["u"], w["w_fc2"], w["b_fc2"]))
    # a few per cent from the exact block, and further from it than the two-product form
    exact = O.block_forward(x, cond, w, heads, 1e-6)
    e4, e2 = O.error_metric(y, exact), O.error_metric(O.block_forward(x, cond, w, heads, 1e-6, fp8=True), exact)
    assert 1e-3 < e4 < 0.3 and e2 < 0.3
    # row subset, stack and packed step are consistent with one another
    rows = np.array([0, 3, 6])
    assert np.allclose(F8.block_forward_fp8(x, cond, w, heads, 1e-6, rows=rows), y[rows], rtol=1e-12, atol=1e-12)
    w2 = _block(rng, H, F, C)
    two = F8.stack_forward_fp8(x, cond, [w, w2], heads, 1e-6)
    assert np.array_equal(two, F8.block_forward_fp8(y, cond, w2, heads, 1e-6))
    packed = np.concatenate([x, x[:3]])
    step = F8.step_forward_fp8(packed, [L, 3], np.stack([cond, cond * 0.5]), [w, w2], heads, 1e-6)
    assert np.array_equal(step[:L], two)
    assert np.array_equal(step[L:], F8.stack_forward_fp8(x[:3], cond * 0.5, [w, w2], heads, 1e-6))


def test_fp8_all_products_is_exact_when_every_operand_sits_on_the_grid():
    """Weights on the e4m3 grid with a column maximum of 448 * 2^k lose nothing; an output projection
    whose left operand rows are on the grid too is then exact, which pins that the scales are removed
    again (a missing or doubled scale would be off by the scale itself)."""
    from oracle import fp8_oracle as F8
    rng = np.random.default_rng(4)
    a = O.quantize_e4m3(rng.uniform(-448, 448, (6, 32))) * 2.0 ** -9
    a[:, 0] = 448.0 * 2.0 ** -9                           # every row's maximum maps to 448 exactly
    w_o = O.quantize_e4m3(rng.uniform(-448, 448, (32, 32))) * 2.0 ** -12
    w_o[0, :] = -448.0 * 2.0 ** -12
    assert np.allclose(O.fp8_linear(a, w_o, np.zeros(32)), a @ w_o, rtol=1e-14, atol=0)


def test_fp8_parallel_block_concatenates_before_it_scales():
    from oracle import fp8_oracle as F8
    rng = np.random.default_rng(5)
    H, F, C, heads, L = 64, 128, 8, 2, 5
    w = {"w_ada": rng.standard_normal((C, 3 * H)) * 0.1, "b_ada": rng.standard_normal(3 * H) * 0.1,
         "w_qkv": rng.standard_normal((H, 3 * H)) * 0.2, "b_qkv": rng.standard_normal(3 * H) * 0.1,
         "w_fc1": rng.standard_normal((H, F)) * 0.2, "b_fc1": rng.standard_normal(F) * 0.1,
         "w_out": rng.standard_normal((H + F, H)) * 0.2, "b_out": rng.standard_normal(H) * 0.1}
    x, cond = rng.standard_normal((L, H)), rng.standard_normal(C)
    t = {}
    y = F8.parallel_block_forward_fp8(x, cond, w, heads, 1e-6, taps=t)
    gate = np.split(O.silu(cond) @ w["w_ada"] + w["b_ada"], 3)[2]
    cat = np.concatenate([t["a"], t["u"]], axis=1)
    assert np.array_equal(y, x + gate * O.fp8_linear(cat, w["w_out"], w["b_out"]))
    # one scale per concatenated row: scaling the attention half by 2^6 changes how the MLP half is rounded
    exact = O.parallel_block_forward(x, cond, w, heads, 1e-6)
    assert 1e-3 < O.error_metric(y, exact) < 0.3
    assert np.array_equal(F8.stack_forward_fp8(x, cond, [w], heads, 1e-6), y)
