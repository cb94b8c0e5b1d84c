"""The seeded input recipe: bf16 rounding, timestep embedding, config shapes."""
import math

import numpy as np

from paper_2510_01565_b200 import workloads as W


def test_bf16_rounding_ties_to_even():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -16, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0], dtype=np.float32)
    bits = W.f32_to_bf16_bits(x)
    assert bits.tolist() == [0x3F80, 0x3F80, 0x3F81, 0x3F82, 0xC020, 0x0000]
    back = W.bf16_to_f64(bits)
    assert back.dtype == np.float64 and back[0] == 1.0 and back[2] == 1.0 + 2.0 ** -7 and back[4] == -2.5
    y = np.random.default_rng(0).standard_normal(1000).astype(np.float32)
    yb = W.bf16_bits_to_f32(W.f32_to_bf16_bits(y))
    assert np.abs(yb - y).max() <= np.abs(y).max() * 2.0 ** -8
    assert (W.f32_to_bf16_bits(yb) == W.f32_to_bf16_bits(y)).all()   # idempotent


def test_timestep_embedding_pins():
    e = W.timestep_embedding(0.0, 8)
    assert e.tolist() == [1, 1, 1, 1, 0, 0, 0, 0]
    t = 123.25
    e = W.timestep_embedding(t, 8)
    assert e[0] == math.cos(t) and e[4] == math.sin(t)                      # frequency 1 first
    assert abs(e[3] - math.cos(t * 10000.0 ** (-3 / 4))) < 1e-15
    assert np.allclose(e[:4] ** 2 + e[4:] ** 2, 1.0)


def test_config_shapes():
    w = W.make_workload("cfg1_small_256", with_weights=True)
    assert w.total_tokens == 256 and w.image_tokens == 256 and w.dims.hidden == 384
    assert w.tokens[0].shape == (256, 384) and w.cond.shape == (1, 384)
    assert w.weights[0]["w_ada"].shape == (384, 6 * 384) and w.weights[0]["w_fc2"].shape == (1536, 384)
    for name, T, img, nb in [("cfg2_512", 1536, 1024, 4), ("cfg3_1024x2", 9216, 8192, 4), ("cfg4_2048", 16896, 16384, 4)]:
        w = W.make_workload(name, with_weights=False)
        assert (w.total_tokens, w.image_tokens, w.n_blocks) == (T, img, nb)
    w = W.make_workload("cfg5_mixed8", with_weights=False)
    assert [r.height for r in w.requests] == [1024, 512, 256, 256, 1024, 2048, 1024, 1024]
    assert w.total_tokens == 38400 and w.image_tokens == 34304 and w.n_blocks == 8
    assert all(0 <= r.timestep < 1000 for r in w.requests)
    assert abs(w.flops_per_step() / 1e12 - 106.34) < 0.01
    assert abs(W.make_workload("cfg3_1024x2", with_weights=False).flops_per_step() / 1e12 - 10.437) < 0.001


def test_seeding_is_reproducible_and_weight_stats():
    a = W.make_workload("cfg1_small_256", seed=0)
    b = W.make_workload("cfg1_small_256", seed=0)
    c = W.make_workload("cfg1_small_256", seed=1)
    assert (a.tokens[0] == b.tokens[0]).all() and (a.weights[0]["w_o"] == b.weights[0]["w_o"]).all()
    assert (a.tokens[0] != c.tokens[0]).any()
    wq = W.bf16_to_f64(a.weights[0]["w_qkv"])
    assert abs(wq.std() - 0.02) < 5e-4 and abs(wq.mean()) < 5e-4
    tok = W.bf16_to_f64(a.tokens[0])
    assert abs(tok.std() - 1.0) < 0.02
