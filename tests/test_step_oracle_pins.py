"""Pins for the oracle of the shell around the block stack (latent -> tokens, timestep ->
conditioning, tokens -> velocity, Euler update).  Each test fixes the oracle against something
other than its own formula: independent index arithmetic, values at special points, identities,
selector weights that reduce a layer to a known map, a closed-form ODE solution.
"""
import math

import numpy as np
import pytest

from oracle import dit_oracle as O
from oracle import step_oracle as S


def test_patchify_against_index_arithmetic():
    # latent value encodes its own coordinates: 10000 c + 100 y + x
    h8, w8 = 6, 10
    z = np.zeros((16, h8, w8))
    for c in range(16):
        for y in range(h8):
            for x in range(w8):
                z[c, y, x] = 10000 * c + 100 * y + x
    tok = S.patchify(z)
    assert tok.shape == (3 * 5, 64)
    for py in range(3):
        for px in range(5):
            row = tok[py * 5 + px]
            for c in range(16):
                for dy in range(2):
                    for dx in range(2):
                        assert row[c * 4 + dy * 2 + dx] == 10000 * c + 100 * (2 * py + dy) + (2 * px + dx)


def test_unpatchify_inverts_patchify():
    rng = np.random.default_rng(0)
    z = rng.standard_normal((16, 8, 12))
    assert np.array_equal(S.unpatchify(S.patchify(z), 8, 12), z)
    t = rng.standard_normal((4 * 6, 64))
    assert np.array_equal(S.patchify(S.unpatchify(t, 8, 12)), t)


def test_token_count_matches_the_packer():
    for (h, w) in [(256, 256), (512, 256), (1024, 2048)]:
        z = np.zeros(S.latent_shape(h, w))
        assert S.patchify(z).shape[0] == O.image_tokens(h, w)


def test_pos_embed_special_points_and_identity():
    hidden = 32                        # 16 per axis: 8 sin + 8 cos
    pe = S.pos_embed_2d(3, 5, hidden)
    assert pe.shape == (15, hidden)
    # token (0, 0): every sine is 0, every cosine is 1
    assert np.array_equal(pe[0], np.concatenate([np.zeros(8), np.ones(8), np.zeros(8), np.ones(8)]))
    # k = 0 has frequency 1: row part sin(py), column part sin(px)
    for py in range(3):
        for px in range(5):
            row = pe[py * 5 + px]
            assert row[0] == pytest.approx(math.sin(py), abs=1e-15)
            assert row[8] == pytest.approx(math.cos(py), abs=1e-15)
            assert row[16] == pytest.approx(math.sin(px), abs=1e-15)
            assert row[24] == pytest.approx(math.cos(px), abs=1e-15)
            # last frequency of each axis: 10000^(-7/8)
            assert row[7] == pytest.approx(math.sin(py * 10000 ** (-7 / 8)), abs=1e-15)
            assert row[23] == pytest.approx(math.sin(px * 10000 ** (-7 / 8)), abs=1e-15)
    # unit circle: sin^2 + cos^2 = 1 for every (token, axis, frequency)
    for a in (0, 16):
        assert np.allclose(pe[:, a:a + 8] ** 2 + pe[:, a + 8:a + 16] ** 2, 1.0, atol=1e-14)
    # the row part does not depend on the column and vice versa
    assert np.array_equal(pe[0 * 5 + 2, :16], pe[0 * 5 + 4, :16])
    assert np.array_equal(pe[1 * 5 + 3, 16:], pe[2 * 5 + 3, 16:])


def test_timestep_embedding_special_points():
    e0 = S.timestep_embedding(0.0)
    assert e0.shape == (256,)
    assert np.array_equal(e0, np.concatenate([np.ones(128), np.zeros(128)]))   # cos half, then sin half
    e = S.timestep_embedding(2.5)
    assert e[0] == pytest.approx(math.cos(2.5), abs=1e-15) and e[128] == pytest.approx(math.sin(2.5), abs=1e-15)
    assert e[127] == pytest.approx(math.cos(2.5 * 10000 ** (-127 / 128)), abs=1e-15)
    assert np.allclose(e[:128] ** 2 + e[128:] ** 2, 1.0, atol=1e-14)
    # t = pi at frequency 1
    e = S.timestep_embedding(math.pi)
    assert e[0] == pytest.approx(-1.0, abs=1e-15) and e[128] == pytest.approx(0.0, abs=1e-15)


def _selector_shell(hidden, cond_dim):
    w = {"w_in": np.zeros((64, hidden)), "b_in": np.zeros(hidden),
         "w_t1": np.zeros((256, cond_dim)), "b_t1": np.zeros(cond_dim),
         "w_t2": np.zeros((cond_dim, cond_dim)), "b_t2": np.zeros(cond_dim),
         "w_fa": np.zeros((cond_dim, 2 * hidden)), "b_fa": np.zeros(2 * hidden),
         "w_out": np.zeros((hidden, 64)), "b_out": np.zeros(64)}
    return w


def test_embed_with_identity_weights_is_patch_plus_position():
    rng = np.random.default_rng(1)
    z = rng.standard_normal((16, 4, 6))
    w = _selector_shell(64, 8)
    w["w_in"] = np.eye(64)
    w["b_in"] = np.full(64, 0.25)
    tok = S.embed_latent(z, w, 64)
    # subtract the position term, checked above, and the bias: what is left is the patch itself
    left = tok - S.pos_embed_2d(2, 3, 64) - 0.25
    assert np.allclose(left, S.patchify(z), atol=1e-15)
    # a transposed weight would fail this: weight row k feeds channel k only
    w["w_in"] = np.zeros((64, 64)); w["w_in"][3, 10] = 2.0
    tok = S.embed_latent(z, w, 64) - S.pos_embed_2d(2, 3, 64) - 0.25
    assert np.allclose(tok[:, 10], 2.0 * S.patchify(z)[:, 3], atol=1e-15)
    assert np.allclose(np.delete(tok, 10, axis=1), 0.0, atol=1e-15)


def test_timestep_cond_hand_case():
    # one active path: e[0] = cos(t) -> hidden unit 2 -> output unit 5
    w = _selector_shell(64, 8)
    w["w_t1"][0, 2] = 3.0
    w["b_t1"][2] = 0.5
    w["w_t2"][2, 5] = -2.0
    w["b_t2"][:] = 0.125
    t = 0.75
    pre = 3.0 * math.cos(t) + 0.5
    want = np.full(8, 0.125)
    want[5] += -2.0 * pre / (1.0 + math.exp(-pre))
    got = S.timestep_cond(t, None, w)
    assert np.allclose(got, want, atol=1e-15)
    pooled = np.arange(8, dtype=np.float64)
    assert np.allclose(S.timestep_cond(t, pooled, w), want + pooled, atol=1e-15)


def test_final_layer_reduces_to_layernorm_and_to_modulation():
    rng = np.random.default_rng(2)
    hidden, cond_dim = 64, 8
    x = rng.standard_normal((5, hidden)) * 3.0 + 1.0
    cond = rng.standard_normal(cond_dim)
    w = _selector_shell(hidden, cond_dim)
    w["w_out"] = np.eye(hidden)[:, :64]
    # zero modulation weights: v_tok = LN(x), rows with zero mean and unit variance
    v = S.final_layer(x, cond, w, 0.0)
    assert np.allclose(v.mean(axis=1), 0.0, atol=1e-14)
    assert np.allclose((v ** 2).mean(axis=1), 1.0, atol=1e-13)
    assert np.allclose(v, (x - x.mean(1, keepdims=True)) / x.std(1, keepdims=True), atol=1e-13)
    # bias-only modulation: shift is the first half, scale the second
    w["b_fa"][:hidden] = 0.5
    w["b_fa"][hidden:] = 1.0
    v2 = S.final_layer(x, cond, w, 0.0)
    assert np.allclose(v2, 2.0 * v + 0.5, atol=1e-13)
    # the cond path: SiLU(cond[1]) scaled into the shift of channel 7 only
    w["b_fa"][:] = 0.0
    w["w_fa"][1, 7] = 4.0
    v3 = S.final_layer(x, cond, w, 0.0)
    s = cond[1] / (1.0 + math.exp(-cond[1]))
    assert np.allclose(v3[:, 7], v[:, 7] + 4.0 * s, atol=1e-13)
    assert np.allclose(np.delete(v3, 7, axis=1), np.delete(v, 7, axis=1), atol=1e-13)
    # output bias and a non-square selector
    w["w_fa"][:] = 0.0
    w["w_out"] = np.zeros((hidden, 64)); w["w_out"][9, 0] = -1.0
    w["b_out"][:] = 0.75
    v4 = S.final_layer(x, cond, w, 0.0)
    assert np.allclose(v4[:, 0], 0.75 - v[:, 9], atol=1e-13)
    assert np.allclose(v4[:, 1:], 0.75, atol=1e-15)


def test_euler_solves_the_straight_line_flow_exactly():
    # Rectified flow with a perfect model: z(sigma) = x0 + sigma * (z1 - x0), velocity (z - x0) / sigma.
    # Explicit Euler is exact on it for any step sizes, and lands on x0 at sigma = 0.
    rng = np.random.default_rng(3)
    x0, noise = rng.standard_normal((16, 4, 4)), rng.standard_normal((16, 4, 4))
    sigmas = [1.0, 0.8, 0.55, 0.3, 0.1, 0.0]
    z = x0 + sigmas[0] * (noise - x0)
    for s, s_next in zip(sigmas[:-1], sigmas[1:]):
        v = (z - x0) / s
        z = S.euler_update(z, v, s_next - s)
        assert np.allclose(z, x0 + s_next * (noise - x0), atol=1e-14)
    assert np.allclose(z, x0, atol=1e-14)


def test_round_to_bf16():
    # exactly representable values stay; ties go to even; 8 significant bits survive
    vals = np.array([1.0, -2.5, 0.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, 3.14159])
    got = S.round_to_bf16(vals)
    assert got[0] == 1.0 and got[1] == -2.5 and got[2] == 0.0
    assert got[3] == 1.0                     # tie between 1 and 1 + 2^-7: even mantissa wins
    assert got[4] == 1.0 + 2 ** -6           # tie between 1 + 2^-7 and 1 + 2^-6: even wins
    assert got[5] == 1.0 + 2 ** -7
    assert got[6] == 3.140625


def test_zero_output_layer_moves_the_latent_by_its_bias():
    # adaLN-Zero style initialisation of the output projection: velocity = b_out per patch entry,
    # whatever the blocks compute; the latent moves by dsigma * b_out.
    rng = np.random.default_rng(4)
    hidden, cond_dim, heads = 64, 8, 1
    w = _selector_shell(hidden, cond_dim)
    w["w_in"] = rng.standard_normal((64, hidden)) * 0.1
    w["w_t1"] = rng.standard_normal((256, cond_dim)) * 0.02
    w["w_t2"] = rng.standard_normal((cond_dim, cond_dim)) * 0.1
    w["b_out"] = np.arange(64, dtype=np.float64) / 64.0
    blk = {"w_ada": rng.standard_normal((cond_dim, 6 * hidden)) * 0.1, "b_ada": np.zeros(6 * hidden),
           "w_qkv": rng.standard_normal((hidden, 3 * hidden)) * 0.1, "b_qkv": np.zeros(3 * hidden),
           "w_o": rng.standard_normal((hidden, hidden)) * 0.1, "b_o": np.zeros(hidden),
           "w_fc1": rng.standard_normal((hidden, 128)) * 0.1, "b_fc1": np.zeros(128),
           "w_fc2": rng.standard_normal((128, hidden)) * 0.1, "b_fc2": np.zeros(hidden)}
    z = rng.standard_normal((16, 4, 8))
    txt = S.round_to_bf16(rng.standard_normal((3, hidden)))
    new, vel, taps = S.denoise_step([z], [txt], [500.0], [-0.02], [None], w, [blk], heads, 1e-6)
    want_v = S.unpatchify(np.tile(w["b_out"], (2 * 4, 1)), 4, 8)
    assert np.allclose(vel[0], want_v, atol=1e-15)
    assert np.allclose(new[0], z - 0.02 * want_v, atol=1e-15)
    assert taps[0]["tokens"].shape == (8 + 3, hidden)
    assert np.array_equal(taps[0]["tokens"][8:], txt)          # text rows follow the image rows unchanged
    assert np.array_equal(taps[0]["tokens"], S.round_to_bf16(taps[0]["tokens"]))


def test_requests_do_not_see_each_other():
    rng = np.random.default_rng(5)
    hidden, cond_dim, heads = 64, 8, 1
    w = {k: rng.standard_normal(v.shape) * 0.1 for k, v in _selector_shell(hidden, cond_dim).items()}
    blk = {"w_ada": rng.standard_normal((cond_dim, 6 * hidden)) * 0.1, "b_ada": rng.standard_normal(6 * hidden) * 0.1,
           "w_qkv": rng.standard_normal((hidden, 3 * hidden)) * 0.1, "b_qkv": np.zeros(3 * hidden),
           "w_o": rng.standard_normal((hidden, hidden)) * 0.1, "b_o": np.zeros(hidden),
           "w_fc1": rng.standard_normal((hidden, 128)) * 0.1, "b_fc1": np.zeros(128),
           "w_fc2": rng.standard_normal((128, hidden)) * 0.1, "b_fc2": np.zeros(hidden)}
    za, zb = rng.standard_normal((16, 4, 4)), rng.standard_normal((16, 2, 6))
    e = np.zeros((0, hidden))
    both, _, _ = S.denoise_step([za, zb], [e, e], [100.0, 900.0], [-0.1, -0.05], [None, None], w, [blk], heads, 1e-6)
    only_b, _, _ = S.denoise_step([zb], [e], [900.0], [-0.05], [None], w, [blk], heads, 1e-6)
    assert np.array_equal(both[1], only_b[0])
