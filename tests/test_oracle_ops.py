"""Pins for the oracle's elementary operations: closed forms and special cases that the
mathematics fixes, chosen so that a dropped term, a wrong sign or index, or a transposed
operand fails at least one of them.  CPU only."""
import math

import numpy as np
import pytest

from oracle import ls_oracle as O
from paper_2404_16710_b200.synth import bf16_bits, bf16_values

ONE = bf16_bits(np.ones(1))[0]


def ones(n):
    return np.full(n, ONE, dtype=np.uint16)


# ---------------------------------------------------------------- RMSNorm
def test_rmsnorm_constant_vector_closed_form():
    c, eps = 3.0, 1e-5
    g = bf16_bits(np.array([1.0, 0.5, 2.0, -1.0, 0.25, 4.0]))
    y = O.rmsnorm(np.full(6, c), g, eps)
    np.testing.assert_allclose(y, bf16_values(g) * c / math.sqrt(c * c + eps), rtol=1e-14)


def test_rmsnorm_three_four():
    eps = 1e-5
    y = O.rmsnorm(np.array([3.0, 4.0]), ones(2), eps)
    np.testing.assert_allclose(y, np.array([3.0, 4.0]) / math.sqrt(12.5 + eps), rtol=1e-14)


def test_rmsnorm_mean_not_sum_and_eps_inside_sqrt():
    # with x = 0 except one entry, mean x^2 = a^2 / D; eps dominates when a is tiny
    D, eps = 8, 1e-2
    x = np.zeros(D)
    x[3] = 1e-6
    y = O.rmsnorm(x, ones(D), eps)
    assert y[3] == pytest.approx(1e-6 / math.sqrt(1e-12 / D + eps), rel=1e-13)
    x[3] = 2.0
    y = O.rmsnorm(x, ones(D), 0.0)
    assert y[3] == pytest.approx(math.sqrt(D), rel=1e-14)  # a / sqrt(a^2 / D)


def test_rmsnorm_scale_invariance():
    rng = np.random.default_rng(0)
    x = rng.normal(size=64)
    g = bf16_bits(1 + 0.1 * rng.normal(size=64))
    np.testing.assert_allclose(O.rmsnorm(x, g, 0.0), O.rmsnorm(1000 * x, g, 0.0), rtol=1e-12)


# ---------------------------------------------------------------- RoPE
def test_rope_position_zero_is_identity():
    v = np.random.default_rng(1).normal(size=16)
    np.testing.assert_array_equal(O.rope(v, 0, 1e4), v)


def test_rope_preserves_norm_per_pair():
    v = np.random.default_rng(2).normal(size=32)
    r = O.rope(v, 77, 1e4)
    np.testing.assert_allclose(r[:16] ** 2 + r[16:] ** 2, v[:16] ** 2 + v[16:] ** 2, rtol=1e-12)


def test_rope_pair_zero_rotates_by_position_radians():
    hd, p = 8, 3
    v = np.zeros(hd)
    v[0] = 1.0  # pair (0, hd/2), frequency theta^0 = 1
    r = O.rope(v, p, 1e4)
    assert r[0] == pytest.approx(math.cos(p), abs=1e-15)
    assert r[hd // 2] == pytest.approx(math.sin(p), abs=1e-15)  # counter-clockwise
    assert np.all(r[[1, 2, 3, 5, 6, 7]] == 0)


def test_rope_frequency_of_every_pair():
    hd, p, theta = 16, 5, 500.0
    for j in range(hd // 2):
        v = np.zeros(hd)
        v[j + hd // 2] = 1.0
        r = O.rope(v, p, theta)
        ang = p * theta ** (-2.0 * j / hd)
        assert r[j] == pytest.approx(-math.sin(ang), abs=1e-14)
        assert r[j + hd // 2] == pytest.approx(math.cos(ang), abs=1e-14)


def test_rope_inner_product_depends_on_relative_position_only():
    rng = np.random.default_rng(3)
    q, k = rng.normal(size=32), rng.normal(size=32)
    a = O.rope(q, 10, 1e4) @ O.rope(k, 4, 1e4)
    b = O.rope(q, 106, 1e4) @ O.rope(k, 100, 1e4)
    assert a == pytest.approx(b, rel=1e-10)


# ---------------------------------------------------------------- softmax / attention
def test_softmax_zero_and_log_three():
    np.testing.assert_allclose(O.softmax([0.0, math.log(3.0)]), [0.25, 0.75], rtol=1e-14)


def test_softmax_shift_invariance_and_large_scores():
    s = np.array([1.0, -2.0, 0.5, 3.0])
    np.testing.assert_allclose(O.softmax(s + 1000.0), O.softmax(s), rtol=1e-12)
    assert np.isfinite(O.softmax(s + 1e4)).all()


def test_attention_single_key_returns_its_value():
    rng = np.random.default_rng(4)
    Hq, Hkv, hd = 4, 2, 8
    q = rng.normal(size=Hq * hd)
    k, v = rng.normal(size=(1, Hkv * hd)), rng.normal(size=(1, Hkv * hd))
    o = O.attention(q, k, v, Hq, Hkv, hd).reshape(Hq, hd)
    vv = v.reshape(Hkv, hd)
    # query head i reads KV head i // (Hq / Hkv)
    np.testing.assert_array_equal(o, vv[[0, 0, 1, 1]])


def test_attention_equal_scores_give_mean_of_values():
    rng = np.random.default_rng(5)
    Hq = Hkv = 2
    hd, n = 4, 5
    v = rng.normal(size=(n, Hkv * hd))
    o = O.attention(rng.normal(size=Hq * hd), np.zeros((n, Hkv * hd)), v, Hq, Hkv, hd)
    np.testing.assert_allclose(o, v.mean(axis=0), rtol=1e-13)


def test_attention_scale_is_one_over_sqrt_head_dim():
    hd = 16
    q = np.zeros(hd)
    q[0] = 1.0
    k = np.zeros((2, hd))
    k[1, 0] = math.log(3.0) * math.sqrt(hd)  # score = ln 3 after the 1/sqrt(hd) scale
    v = np.zeros((2, hd))
    v[0, 0], v[1, 0] = 1.0, 5.0
    o = O.attention(q, k, v, 1, 1, hd)
    assert o[0] == pytest.approx(0.25 * 1.0 + 0.75 * 5.0, rel=1e-13)


def test_attention_matches_numpy_definition():
    rng = np.random.default_rng(6)
    Hq, Hkv, hd, n = 6, 3, 8, 11
    q = rng.normal(size=Hq * hd)
    k, v = rng.normal(size=(n, Hkv * hd)), rng.normal(size=(n, Hkv * hd))
    o = O.attention(q, k, v, Hq, Hkv, hd).reshape(Hq, hd)
    for i in range(Hq):
        kh = i // (Hq // Hkv)
        s = k[:, kh * hd:(kh + 1) * hd] @ q[i * hd:(i + 1) * hd] / math.sqrt(hd)
        a = np.exp(s - s.max())
        a /= a.sum()
        np.testing.assert_allclose(o[i], a @ v[:, kh * hd:(kh + 1) * hd], rtol=1e-12)


# ---------------------------------------------------------------- SiLU, linear, argmax, match
def test_silu_identities():
    assert O.silu(0.0) == 0.0
    for z in (0.3, 2.0, 7.5):
        assert O.silu(z) - O.silu(-z) == pytest.approx(z, rel=1e-14)
    assert O.silu(math.log(3.0)) == pytest.approx(0.75 * math.log(3.0), rel=1e-14)


def test_linear_is_row_major_matrix_vector_product():
    rng = np.random.default_rng(7)
    W = bf16_bits(rng.normal(size=(5, 9)))  # not square: a transposed read cannot pass
    h = rng.normal(size=9)
    np.testing.assert_allclose(O.linear(W, h), bf16_values(W) @ h, rtol=1e-13)
    # a one-hot input picks a column
    e = np.zeros(9)
    e[2] = 1.0
    np.testing.assert_array_equal(O.linear(W, e), bf16_values(W)[:, 2])


def test_argmax_lowest_index_wins_ties_and_margin():
    i, mg, ma = O.argmax([1.0, 5.0, 5.0, -7.0])
    assert (i, mg, ma) == (1, 0.0, 7.0)
    i, mg, _ = O.argmax([0.5, 2.0, -1.0])
    assert i == 1 and mg == pytest.approx(1.5)


@pytest.mark.parametrize("draft,verified,n", [
    ([5, 6, 7], [9, 6, 7, 1], 0),        # first draft wrong; later agreement must not count
    ([5, 6, 7], [5, 6, 2, 1], 2),
    ([5, 6, 7], [5, 0, 7, 1], 1),
    ([5, 6, 7], [5, 6, 7, 1], 3),        # all accepted; verified[3] is the bonus token
])
def test_match_counts_leading_agreements(draft, verified, n):
    assert O.match(draft, verified) == n
