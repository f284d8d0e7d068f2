"""Pins for the oracle's RMSNorm, projection, key-norm and rotation (no GPU).

Each test checks the oracle against something fixed by the paper or by mathematics, not against
the oracle's own formula: hand-computed values, invariants stated in the paper (degree-0
homogeneity after Eq. 2; orthogonality and position-only dependence of R_p after Eq. 12), a
library matmul in the special case where Eq. 13-14 reduce to one, an explicitly built rotation
matrix, and the closed form of the sliding-window mismatch of Eq. 16.
"""
import math

import numpy as np
import pytest

import oracle
from kvd_synth import (ROPE_HALF, ROPE_INTERLEAVED, SMOLLM2_135M, TINY_GQA, bf16_to_f64, make_layer_weights,
                       make_residuals)


# ------------------------------------------------------------------------------- RMSNorm
def test_rmsnorm_hand_case():
    # x = (3, 4): mean square = 12.5
    out = oracle.rmsnorm([3.0, 4.0], [1.0, 1.0], 0.0)
    assert out[0] == pytest.approx(3.0 / math.sqrt(12.5), rel=1e-15)
    assert out[1] == pytest.approx(4.0 / math.sqrt(12.5), rel=1e-15)
    # gamma multiplies channel-wise
    out = oracle.rmsnorm([3.0, 4.0], [2.0, -0.5], 0.0)
    assert out[0] == pytest.approx(6.0 / math.sqrt(12.5), rel=1e-15)
    assert out[1] == pytest.approx(-2.0 / math.sqrt(12.5), rel=1e-15)


def test_rmsnorm_eps_inside_root():
    # x = (1, 1), eps = 3: sqrt(1 + 3) = 2
    out = oracle.rmsnorm([1.0, 1.0], [1.0, 1.0], 3.0)
    assert np.array_equal(out, [0.5, 0.5])


def test_rmsnorm_degree_zero_homogeneity_bit_exact():
    # scaling by a power of two is exact in binary floating point, so with eps = 0 the
    # statement RMSNorm(a x) = RMSNorm(x) must hold to the last bit
    rng = np.random.default_rng(1)
    x = rng.standard_normal(576)
    g = 1.0 + 0.02 * rng.standard_normal(576)
    base = oracle.rmsnorm(x, g, 0.0)
    for k in (-7, -1, 3, 10):
        assert np.array_equal(oracle.rmsnorm(x * 2.0 ** k, g, 0.0), base)
    # and approximately for any positive factor
    np.testing.assert_allclose(oracle.rmsnorm(x * 3.7, g, 0.0), base, rtol=1e-14)


def test_rmsnorm_unit_rms():
    rng = np.random.default_rng(2)
    x = rng.standard_normal(2560) * 5
    g = 1.0 + 0.02 * rng.standard_normal(2560)
    y = oracle.rmsnorm(x, g, 0.0) / g
    assert math.sqrt(np.mean(y * y)) == pytest.approx(1.0, rel=1e-14)


# ------------------------------------------------------------------------------- RoPE
def _rotation_matrix(d, pos, theta, style):
    """R_p built entry by entry from the text after Eq. 12 (block-diagonal 2x2 rotations)."""
    R = np.zeros((d, d))
    for i in range(d // 2):
        phi = pos * theta ** (-2.0 * i / d)
        a, b = (2 * i, 2 * i + 1) if style == ROPE_INTERLEAVED else (i, i + d // 2)
        R[a, a] = math.cos(phi)
        R[a, b] = -math.sin(phi)
        R[b, a] = math.sin(phi)
        R[b, b] = math.cos(phi)
    return R


@pytest.mark.parametrize("style", [ROPE_INTERLEAVED, ROPE_HALF])
def test_rope_matches_explicit_matrix(style):
    rng = np.random.default_rng(3)
    x = rng.standard_normal(64)
    for pos in (0, 1, 7, 511, 32767):
        R = _rotation_matrix(64, pos, 1.0e4, style)
        np.testing.assert_allclose(oracle.rope(x, pos, 1.0e4, style), R @ x, atol=1e-13)
        # orthogonality stated after Eq. 12
        np.testing.assert_allclose(R.T @ R, np.eye(64), atol=1e-13)


@pytest.mark.parametrize("style", [ROPE_INTERLEAVED, ROPE_HALF])
def test_rope_identity_norm_and_composition(style):
    rng = np.random.default_rng(4)
    x = rng.standard_normal(128)
    assert np.array_equal(oracle.rope(x, 0, 1.0e6, style), x)  # R_0 = I
    for p in (1, 100, 4095):
        y = oracle.rope(x, p, 1.0e6, style)
        assert np.linalg.norm(y) == pytest.approx(np.linalg.norm(x), rel=1e-14)
    # R_p R_q = R_{p+q}
    y = oracle.rope(oracle.rope(x, 37, 1.0e4, style), 1000, 1.0e4, style)
    np.testing.assert_allclose(y, oracle.rope(x, 1037, 1.0e4, style), atol=1e-12)


def test_rope_first_and_last_frequency():
    d, theta = 64, 1.0e4
    e = np.zeros(d)
    e[0] = 1.0  # first pair, interleaved: rotates by exactly pos * 1 rad
    y = oracle.rope(e, 1, theta, ROPE_INTERLEAVED)
    assert y[0] == pytest.approx(math.cos(1.0), abs=1e-16)
    assert y[1] == pytest.approx(math.sin(1.0), abs=1e-16)
    assert np.all(y[2:] == 0.0)
    e = np.zeros(d)
    e[d - 2] = 1.0  # last pair: angle theta^(-(d-2)/d)
    phi = theta ** (-(d - 2) / d)
    y = oracle.rope(e, 1, theta, ROPE_INTERLEAVED)
    assert y[d - 2] == pytest.approx(math.cos(phi), abs=1e-16)
    assert y[d - 1] == pytest.approx(math.sin(phi), abs=1e-16)
    # sign convention of Eq. 11-12: second channel of a pair feeds the first with a minus sign
    e = np.zeros(d)
    e[1] = 1.0
    y = oracle.rope(e, 1, theta, ROPE_INTERLEAVED)
    assert y[0] == pytest.approx(-math.sin(1.0), abs=1e-16)
    assert y[1] == pytest.approx(math.cos(1.0), abs=1e-16)


def test_rope_styles_differ_by_a_channel_permutation():
    # HALF is INTERLEAVED seen through the permutation (2i -> i, 2i+1 -> i + d/2)
    d = 64
    rng = np.random.default_rng(5)
    x = rng.standard_normal(d)
    perm = np.empty(d, dtype=int)
    perm[: d // 2] = np.arange(0, d, 2)
    perm[d // 2:] = np.arange(1, d, 2)
    y_int = oracle.rope(x, 123, 1.0e4, ROPE_INTERLEAVED)
    y_half = oracle.rope(x[perm], 123, 1.0e4, ROPE_HALF)
    np.testing.assert_allclose(y_half, y_int[perm], atol=1e-14)


def test_sliding_window_mismatch_closed_form():
    # Eq. 16: ||(R_j - R_{j-w}) k||^2 = sum_i 4 sin^2(w phi_i / 2) (a_i^2 + b_i^2), zero iff w = 0
    d, theta, j = 64, 1.0e4, 700
    rng = np.random.default_rng(6)
    k = rng.standard_normal(d)
    for w in (0, 1, 5, 256):
        diff = oracle.rope(k, j, theta) - oracle.rope(k, j - w, theta)
        expect = 0.0
        for i in range(d // 2):
            phi = theta ** (-2.0 * i / d)
            expect += 4.0 * math.sin(w * phi / 2.0) ** 2 * (k[2 * i] ** 2 + k[2 * i + 1] ** 2)
        assert float(diff @ diff) == pytest.approx(expect, rel=1e-10, abs=1e-20)
        if w == 0:
            assert np.all(diff == 0.0)
        else:
            assert np.linalg.norm(diff) > 1e-3


# ------------------------------------------------------------------------------- projection
def test_projection_hand_case():
    # d_hidden = 2, one KV head of d_head = 2, gamma = 1, eps = 0, position 0 (no rotation)
    # x = (3, 4) -> xbar = (3, 4)/sqrt(12.5); W_K = [[1, 2], [3, 4]], W_V = [[5, 6], [7, 8]]
    X = np.array([[3.0, 4.0]])
    W = np.array([[1.0, 2.0, 5.0, 6.0], [3.0, 4.0, 7.0, 8.0]])
    K, V = oracle.recompute_kv(X, [0], [1.0, 1.0], W, 1, 2, 0.0, 1.0e4)
    r = math.sqrt(12.5)
    np.testing.assert_allclose(K[0, 0], [(3 * 1 + 4 * 3) / r, (3 * 2 + 4 * 4) / r], rtol=1e-15)
    np.testing.assert_allclose(V[0, 0], [(3 * 5 + 4 * 7) / r, (3 * 6 + 4 * 8) / r], rtol=1e-15)
    # position 1: the key pair rotates by 1 rad, the value does not move
    K1, V1 = oracle.recompute_kv(X, [1], [1.0, 1.0], W, 1, 2, 0.0, 1.0e4)
    a, b = K[0, 0]
    np.testing.assert_allclose(K1[0, 0], [a * math.cos(1) - b * math.sin(1), a * math.sin(1) + b * math.cos(1)],
                               rtol=1e-14)
    assert np.array_equal(V1, V)


def test_projection_reduces_to_library_matmul():
    # no key-norm, positions 0: K = RMSNorm(X) W_K, V = RMSNorm(X) W_V  -> numpy matmul
    s = SMOLLM2_135M
    w = make_layer_weights(s)
    X = bf16_to_f64(make_residuals(s, 37, seed=11))
    W = bf16_to_f64(w.w_kv)
    g = bf16_to_f64(w.gamma_in)
    K, V = oracle.recompute_kv(X, np.zeros(37, np.int32), g, W, s.n_kv_heads, s.d_head, s.rms_eps, s.rope_theta)
    Xb = X / np.sqrt(np.mean(X * X, axis=1, keepdims=True) + s.rms_eps) * g
    ref = Xb @ W
    kvd = s.n_kv_heads * s.d_head
    np.testing.assert_allclose(K.reshape(37, kvd), ref[:, :kvd], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(V.reshape(37, kvd), ref[:, kvd:], rtol=1e-12, atol=1e-13)


def test_head_layout_and_kv_split():
    # W_K routes input channel c to key channel c of head (c // d_head); W_V routes it doubled.
    # A transposed weight, swapped K/V halves or a wrong head stride would all fail here.
    d_hidden, n_kv, d_head = 8, 2, 4
    W = np.zeros((d_hidden, 2 * n_kv * d_head))
    for c in range(d_hidden):
        W[c, c] = 1.0
        W[c, n_kv * d_head + c] = 2.0
    W[0, 5] = 10.0  # asymmetric entry: input 0 also feeds head 1, channel 1 of K
    x = np.arange(1.0, 9.0)[None, :]
    K, V = oracle.recompute_kv(x, [0], np.ones(8), W, n_kv, d_head, 0.0, 1.0e4)
    xb = x[0] / math.sqrt(np.mean(x * x))
    expK = xb.reshape(2, 4).copy()
    expK[1, 1] += 10.0 * xb[0]
    np.testing.assert_allclose(K[0], expK, rtol=1e-15)
    np.testing.assert_allclose(V[0], 2.0 * xb.reshape(2, 4), rtol=1e-15)


def test_rows_are_independent_and_order_free():
    # Prop. 3.2's premise: a row's K/V depend on that row and its position only -> bit-equal
    # whether the row is computed alone, in a batch, or at another batch index.
    s = TINY_GQA
    w = make_layer_weights(s)
    X = bf16_to_f64(make_residuals(s, 9, seed=12))
    pos = np.array([5, 0, 77, 3, 1000, 8, 9, 10, 4095], np.int32)
    args = (bf16_to_f64(w.gamma_in), bf16_to_f64(w.w_kv), s.n_kv_heads, s.d_head, s.rms_eps, s.rope_theta,
            bf16_to_f64(w.gamma_k), s.rms_eps)
    K, V = oracle.recompute_kv(X, pos, *args)
    for m in (0, 4, 8):
        k1, v1 = oracle.recompute_kv(X[m:m + 1], pos[m:m + 1], *args)
        assert np.array_equal(k1[0], K[m]) and np.array_equal(v1[0], V[m])
    perm = np.random.default_rng(0).permutation(9)
    Kp, Vp = oracle.recompute_kv(X[perm], pos[perm], *args)
    assert np.array_equal(Kp, K[perm]) and np.array_equal(Vp, V[perm])


# ------------------------------------------------------------------------------- key norm
def test_key_norm_hand_case():
    # identity projection, d_head = 2: k_raw = xbar = (3,4)/sqrt(12.5) -> key-norm -> (3,4)/sqrt(12.5) again
    # (the norm of an already unit-RMS vector is itself), times gamma_k = (2, 0.5)
    W = np.array([[1.0, 0.0, 0.0, 0.0], [0.0, 1.0, 0.0, 0.0]])
    K, V = oracle.recompute_kv([[3.0, 4.0]], [0], [1.0, 1.0], W, 1, 2, 0.0, 1.0e4, gamma_k=[2.0, 0.5], qk_eps=0.0)
    r = math.sqrt(12.5)
    np.testing.assert_allclose(K[0, 0], [2.0 * 3 / r, 0.5 * 4 / r], rtol=1e-14)
    assert np.all(V == 0.0)


def test_key_norm_is_per_head_before_rotation_and_scale_free():
    s = TINY_GQA
    w = make_layer_weights(s)
    X = bf16_to_f64(make_residuals(s, 5, seed=13))
    W = bf16_to_f64(w.w_kv)
    g = bf16_to_f64(w.gamma_in)
    ones = np.ones(s.d_head)
    pos = np.array([0, 1, 50, 1000, 9], np.int32)
    K, V = oracle.recompute_kv(X, pos, g, W, s.n_kv_heads, s.d_head, s.rms_eps, s.rope_theta, ones, 0.0)
    # with gamma_k = 1 and eps = 0 every head has RMS exactly 1; the rotation keeps the norm
    rms = np.sqrt(np.mean(K * K, axis=2))
    np.testing.assert_allclose(rms, 1.0, rtol=1e-13)
    # scaling W_K by a power of two cannot change a normalised key; V doubles
    W2 = W.copy()
    kvd = s.n_kv_heads * s.d_head
    W2[:, :kvd] *= 4.0
    W2[:, kvd:] *= 2.0
    K2, V2 = oracle.recompute_kv(X, pos, g, W2, s.n_kv_heads, s.d_head, s.rms_eps, s.rope_theta, ones, 0.0)
    assert np.array_equal(K2, K)
    assert np.array_equal(V2, 2.0 * V)
    # norm happens before the rotation: un-rotating gives gamma_k-scaled unit-RMS vectors
    gk = bf16_to_f64(w.gamma_k)
    K3, _ = oracle.recompute_kv(X, pos, g, W, s.n_kv_heads, s.d_head, s.rms_eps, s.rope_theta, gk, 0.0)
    for m in range(5):
        for h in range(s.n_kv_heads):
            unrot = oracle.rope(K3[m, h], -int(pos[m]), s.rope_theta)
            np.testing.assert_allclose(unrot / gk, oracle.rope(K[m, h], -int(pos[m]), s.rope_theta), atol=1e-12)
