"""Pins for the CPU oracle: closed forms, hand-derived cases, invariants, brute force.

None of these compares the oracle with the CUDA path; they fix the oracle to
the mathematics and to the numbers the paper prints (Table 1 token counts).
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import dit_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_weights(rng, H, F, C, std=0.3):
    shp = {"w_ada": (C, 6 * H), "b_ada": (6 * H,), "w_qkv": (H, 3 * H), "b_qkv": (3 * H,),
           "w_o": (H, H), "b_o": (H,), "w_fc1": (H, F), "b_fc1": (F,), "w_fc2": (F, H), "b_fc2": (H,)}
    return {k: rng.standard_normal(s) * std for k, s in shp.items()}


# ---------------------------------------------------------------- packer
def test_token_counts_match_table1():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table1_tokens.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 4
    for h, w, n in rows:
        assert O.image_tokens(int(h), int(w)) == int(n)


def test_packer_maps_brute_force():
    reqs = [(256, 256, 0), (512, 256, 7), (16, 16, 0), (1024, 1024, 512), (32, 48, 1)]
    lens, cu, row_req, row_local = O.pack_requests(reqs)
    assert lens.tolist() == [256, 512 + 7, 1, 4096 + 512, 6 + 1]
    assert cu[0] == 0 and cu[-1] == lens.sum() == len(row_req) == len(row_local)
    assert lens.dtype == cu.dtype == row_req.dtype == row_local.dtype == np.int32
    for p in range(cu[-1]):                       # inverse map, row by row
        r = row_req[p]
        assert cu[r] <= p < cu[r + 1] and cu[r] + row_local[p] == p
    assert (np.diff(cu) == lens).all()


def test_packer_special_cases():
    lens, cu, rr, rl = O.pack_requests([(256, 256, 0)])
    assert lens.tolist() == [256] and cu.tolist() == [0, 256] and (rr == 0).all() and rl.tolist() == list(range(256))
    lens, cu, rr, rl = O.pack_requests([])
    assert lens.size == 0 and cu.tolist() == [0] and rr.size == 0
    with pytest.raises(ValueError):
        O.image_tokens(250, 256)
    with pytest.raises(ValueError):
        O.pack_requests([(256, 256, -1)])


# ---------------------------------------------------------------- elementwise closed forms
def test_silu_gelu_known_values():
    assert O.silu(np.array([0.0]))[0] == 0.0
    # silu(ln 3) = ln3 / (1 + 1/3) = 3 ln3 / 4
    assert O.silu(np.array([math.log(3.0)]))[0] == pytest.approx(0.75 * math.log(3.0), rel=1e-15)
    assert O.silu(np.array([-math.log(3.0)]))[0] == pytest.approx(-0.25 * math.log(3.0), rel=1e-15)
    g = O.gelu_tanh(np.array([0.0, 1.0, -1.0, 3.0, 40.0, -40.0]))
    assert g[0] == 0.0
    # widely tabulated value of the tanh form at 1 (differs from the erf form's 0.841345)
    assert g[1] == pytest.approx(0.8411919906, abs=1e-9)
    assert g[1] - g[2] == pytest.approx(1.0, abs=1e-15)          # g(z) - g(-z) = z
    assert g[3] == pytest.approx(2.99636, abs=1e-5)
    assert g[4] == 40.0 and g[5] == 0.0


def test_layer_norm_closed_form():
    x = np.array([[1.0, 3.0, 5.0, 7.0]])                      # mean 4, biased var 5
    np.testing.assert_allclose(O.layer_norm(x, 0.0), np.array([[-3, -1, 1, 3]]) / math.sqrt(5.0), rtol=1e-15)
    np.testing.assert_allclose(O.layer_norm(x, 4.0), np.array([[-3, -1, 1, 3]]) / 3.0, rtol=1e-15)
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 64)) * 3 + 2
    eps = 0.5
    y = O.layer_norm(x, eps)
    var = x.var(axis=1)
    np.testing.assert_allclose(y.mean(axis=1), 0, atol=1e-14)
    np.testing.assert_allclose(y.var(axis=1), var / (var + eps), rtol=1e-13)
    assert (O.layer_norm(np.full((2, 8), 7.25), 1e-6) == 0).all()        # constant row -> 0
    # affine invariance: LN(a x + b) = LN(x) when eps = 0, a > 0
    np.testing.assert_allclose(O.layer_norm(3 * x + 11, 0.0), O.layer_norm(x, 0.0), rtol=1e-12, atol=1e-13)


def test_modulation_special_cases_and_order():
    rng = np.random.default_rng(2)
    H, C = 4, 3
    w_ada, b_ada = rng.standard_normal((C, 6 * H)), rng.standard_normal(6 * H)
    parts = O.adaln_modulation(np.zeros(C), w_ada, b_ada)             # SiLU(0)=0 -> bias only
    np.testing.assert_array_equal(np.concatenate(parts), b_ada)
    parts = O.adaln_modulation(rng.standard_normal(C), np.zeros((C, 6 * H)), b_ada)
    np.testing.assert_array_equal(np.concatenate(parts), b_ada)
    # one-hot cond at ln 3: mod = 0.75 ln3 * row + bias; chunk i is columns [iH, (i+1)H)
    c = np.zeros(C); c[1] = math.log(3.0)
    parts = O.adaln_modulation(c, w_ada, b_ada)
    for i in range(6):
        np.testing.assert_allclose(parts[i], 0.75 * math.log(3.0) * w_ada[1, i * H:(i + 1) * H] + b_ada[i * H:(i + 1) * H], rtol=1e-14)
    # modulate = xhat*(1+scale)+shift
    np.testing.assert_array_equal(O.modulate(np.array([2.0, -1.0]), np.array([1.0, 1.0]), np.array([0.5, -1.0])),
                                  np.array([4.0, 1.0]))


# ---------------------------------------------------------------- attention
def test_attention_rows_sum_to_one_and_shift_invariance():
    rng = np.random.default_rng(3)
    s = rng.standard_normal((7, 11)) * 5
    p = O.softmax_rows(s)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, atol=1e-15)
    np.testing.assert_allclose(O.softmax_rows(s + rng.standard_normal((7, 1)) * 10), p, rtol=1e-12)
    # softmax of ln(c_j) is c_j / sum c
    np.testing.assert_allclose(O.softmax_rows(np.log(np.array([[1.0, 2.0, 5.0]]))), [[1 / 8, 2 / 8, 5 / 8]], rtol=1e-15)


def test_attention_special_cases():
    rng = np.random.default_rng(4)
    L, nh, d = 9, 3, 4
    H = nh * d
    q, k, v = (rng.standard_normal((L, H)) for _ in range(3))
    # single token: a = v
    np.testing.assert_allclose(O.attention(q[:1], k[:1], v[:1], nh), v[:1], rtol=1e-15)
    # zero queries: uniform weights -> column mean of v
    np.testing.assert_allclose(O.attention(np.zeros_like(q), k, v, nh), np.tile(v.mean(0), (L, 1)), rtol=1e-13)
    # heads are independent: changing head 2's q/k/v leaves heads 0,1 untouched
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    for t in (q2, k2, v2):
        t[:, 2 * d:] += 1.0
    a, a2 = O.attention(q, k, v, nh), O.attention(q2, k2, v2, nh)
    np.testing.assert_array_equal(a[:, :2 * d], a2[:, :2 * d])
    assert np.abs(a[:, 2 * d:] - a2[:, 2 * d:]).max() > 0.1
    # brute force per (row, head) with scalar loops
    for i in (0, 5):
        for j in range(nh):
            sc = [sum(q[i, j * d + c] * k[t, j * d + c] for c in range(d)) / math.sqrt(d) for t in range(L)]
            e = [math.exp(x) for x in sc]
            for c in range(d):
                want = sum(e[t] * v[t, j * d + c] for t in range(L)) / sum(e)
                assert a[i, j * d + c] == pytest.approx(want, rel=1e-12)
    # row subset and slabs give the same rows
    rows = np.array([7, 2, 2, 0])
    np.testing.assert_allclose(O.attention(q, k, v, nh, rows=rows), a[rows], rtol=1e-14)
    np.testing.assert_allclose(O.attention(q, k, v, nh, slab=4), a, rtol=1e-14)
    # a very dominant key: weights -> one-hot, a -> that key's value
    kk = np.zeros((3, 4)); kk[1] = 50.0
    qq = np.ones((2, 4))
    vv = rng.standard_normal((3, 4))
    np.testing.assert_allclose(O.attention(qq, kk, vv, 1), np.tile(vv[1], (2, 1)), rtol=1e-12)


# ---------------------------------------------------------------- whole block
def _hand_case():
    ln2 = math.log(2.0)
    w = {
        "w_ada": np.zeros((1, 12)),
        "b_ada": np.array([1, 0, 1, 1, 1, 2, 0, 0.5, 0, 1, 2, -1], dtype=np.float64),
        "w_qkv": np.array([[math.sqrt(2.0) * ln2, 0, 1, 0, 1, 0],
                           [0, 0, 0, 0, 0, 1]], dtype=np.float64),
        "b_qkv": np.array([0, 0, 0, 0, 0, 1], dtype=np.float64),
        "w_o": np.array([[1, 1], [0, 1]], dtype=np.float64),
        "b_o": np.array([1, 0], dtype=np.float64),
        "w_fc1": np.array([[1, 0], [0, 2]], dtype=np.float64),
        "b_fc1": np.zeros(2),
        "w_fc2": np.array([[1, -1], [2, 0]], dtype=np.float64),
        "b_fc2": np.array([0, 1], dtype=np.float64),
    }
    x = np.array([[3, 1], [0, 4]], dtype=np.float64)
    return x, np.zeros(1), w


def _golden_rationals():
    out = {}
    for line in open(os.path.join(GOLDEN, "hand_case_2tok.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, *nums = line.split()
        vals = [Fraction(int(nums[i]), int(nums[i + 1])) for i in range(0, len(nums), 2)]
        out[name] = np.array([float(v) for v in vals]).reshape(2, 2)
    return out


def test_hand_derived_two_token_block():
    x, c, w = _hand_case()
    gold = _golden_rationals()
    taps = {}
    y = O.block_forward(x, c, w, n_heads=1, eps=0.0, taps=taps)
    np.testing.assert_allclose(taps["h1"], [[3, -2], [-1, 2]], rtol=1e-15)
    q, k, v = taps["qkv"][:, :2], taps["qkv"][:, 2:4], taps["qkv"][:, 4:]
    np.testing.assert_allclose(O.softmax_rows(q @ k.T / math.sqrt(2.0)), gold["P"], rtol=1e-13)
    np.testing.assert_allclose(v, [[3, -1], [-1, 3]], rtol=1e-15)
    np.testing.assert_allclose(taps["a"], gold["a"], rtol=1e-13)
    np.testing.assert_allclose(taps["x_mid"], gold["x_mid"], rtol=1e-13)
    np.testing.assert_allclose(taps["h2"], [[1, -1.5], [-1, 2.5]], rtol=1e-13)

    def g(z):  # the tanh-form GELU at a scalar
        return 0.5 * z * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (z + 0.044715 * z ** 3)))
    want = np.array([[3 + 16384 / 4097 + 2 * (g(1.0) + 2 * g(-3.0)), 5 - (1 - g(1.0))],
                     [4 / 17 + 2 * (g(-1.0) + 2 * g(5.0)), 8 - (1 - g(-1.0))]])
    np.testing.assert_allclose(y, want, rtol=1e-13)
    # decimal spot value from the tabulated g(1) = 0.8411919906: y01 = 4.8411919906
    assert y[0, 1] == pytest.approx(4.8411919906, abs=1e-9)
    # same case through the scalar-loop and the masked statements
    np.testing.assert_allclose(np.array(O.block_forward_scalar(x.tolist(), c.tolist(), w, 1, 0.0)), want, rtol=1e-13)
    np.testing.assert_allclose(O.step_forward_masked(x, [2], c[None], [w], 1, 0.0), want, rtol=1e-13)


def test_three_codings_agree_on_random_small_block():
    rng = np.random.default_rng(5)
    H, nh, F, C, L = 8, 2, 12, 5, 4
    w = _rand_weights(rng, H, F, C)
    x, c = rng.standard_normal((L, H)), rng.standard_normal(C)
    y = O.block_forward(x, c, w, nh, 1e-6)
    ys = np.array(O.block_forward_scalar(x.tolist(), c.tolist(), w, nh, 1e-6))
    ym = O.step_forward_masked(x, [L], c[None], [w], nh, 1e-6)
    np.testing.assert_allclose(ys, y, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(ym, y, rtol=1e-12, atol=1e-12)


def test_zero_gate_is_identity():
    rng = np.random.default_rng(6)
    H, nh, F, C, L = 16, 4, 32, 16, 10
    blocks = []
    for _ in range(3):
        w = _rand_weights(rng, H, F, C)
        for i in (2, 5):                       # gate_a and gate_m chunks
            w["w_ada"][:, i * H:(i + 1) * H] = 0.0
            w["b_ada"][i * H:(i + 1) * H] = 0.0
        blocks.append(w)
    x, c = rng.standard_normal((L, H)), rng.standard_normal(C)
    np.testing.assert_array_equal(O.stack_forward_alone(x, c, blocks, nh, 1e-6), x)
    # only the MLP gate zero: output equals the attention-branch result
    w = _rand_weights(rng, H, F, C)
    w["w_ada"][:, 5 * H:] = 0.0
    w["b_ada"][5 * H:] = 0.0
    taps = {}
    y = O.block_forward(x, c, w, nh, 1e-6, taps=taps)
    np.testing.assert_array_equal(y, taps["x_mid"])


def test_row_permutation_equivariance():
    rng = np.random.default_rng(7)
    H, nh, F, C, L = 16, 2, 24, 8, 13
    blocks = [_rand_weights(rng, H, F, C) for _ in range(2)]
    x, c = rng.standard_normal((L, H)), rng.standard_normal(C)
    perm = rng.permutation(L)
    y = O.stack_forward_alone(x, c, blocks, nh, 1e-6)
    yp = O.stack_forward_alone(x[perm], c, blocks, nh, 1e-6)
    np.testing.assert_allclose(yp, y[perm], rtol=1e-11, atol=1e-12)


def test_packed_equals_each_request_alone():
    rng = np.random.default_rng(8)
    H, nh, F, C = 16, 2, 24, 8
    lens = [5, 1, 9, 3]
    blocks = [_rand_weights(rng, H, F, C) for _ in range(2)]
    x = rng.standard_normal((sum(lens), H))
    cond = rng.standard_normal((len(lens), C))
    y = O.step_forward(x, lens, cond, blocks, nh, 1e-6)
    ym = O.step_forward_masked(x, lens, cond, blocks, nh, 1e-6)
    np.testing.assert_allclose(ym, y, rtol=1e-11, atol=1e-12)
    p = 0
    for r, l in enumerate(lens):
        alone = O.stack_forward_alone(x[p:p + l], cond[r], blocks, nh, 1e-6)
        np.testing.assert_array_equal(y[p:p + l], alone)
        p += l
    # a request's output does not depend on its neighbours
    x2 = x.copy(); x2[:5] += 1.0
    y2 = O.step_forward(x2, lens, cond, blocks, nh, 1e-6)
    np.testing.assert_array_equal(y2[5:], y[5:])


def test_row_subset_block_matches_full():
    rng = np.random.default_rng(9)
    H, nh, F, C, L = 16, 4, 20, 6, 12
    w = _rand_weights(rng, H, F, C)
    x, c = rng.standard_normal((L, H)), rng.standard_normal(C)
    rows = np.array([11, 0, 4])
    np.testing.assert_allclose(O.block_forward(x, c, w, nh, 1e-6, rows=rows),
                               O.block_forward(x, c, w, nh, 1e-6)[rows], rtol=1e-13, atol=1e-14)


def test_error_metric():
    ref = np.array([[3.0, 4.0]])
    assert O.error_metric(ref + np.array([[0.0, 0.5]]), ref) == pytest.approx(0.5 / math.sqrt(12.5))
