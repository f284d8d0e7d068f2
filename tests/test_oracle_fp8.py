"""Pins of the FP8-checkpoint oracle (CPU only).

  * e4m3_round against the value table that the format's definition implies (all 256 codes decoded from
    their bit fields), against hand-computed ties, and against PyTorch's own float8_e4m3fn conversion on the
    CPU (an independent library routine);
  * quantize_rows / quantize_weights: representable inputs survive unchanged, the scale is max|x| / 448, the
    relative error of a normal value is at most 2^-4;
  * recompute_kv_fp8 reduces to the plain (already pinned) oracle when the inputs are exactly representable,
    and stays within the format's error bound of it otherwise.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import fp8


def decode_e4m3(code: int) -> float:
    """Value of an E4M3 (fn) code from its fields: sign(1) exponent(4, bias 7) mantissa(3); 0x7f / 0xff are NaN."""
    s = -1.0 if code & 0x80 else 1.0
    e, m = (code >> 3) & 0xF, code & 7
    if e == 0xF and m == 7:
        return float("nan")
    if e == 0:
        return s * m * 2.0 ** -9
    return s * (1 + m / 8.0) * 2.0 ** (e - 7)


GRID = np.array(sorted(v for v in (decode_e4m3(c) for c in range(256)) if v == v))


def test_the_grid_has_the_formats_landmarks():
    assert GRID.max() == 448.0 and GRID.min() == -448.0
    pos = GRID[GRID > 0]
    assert pos.min() == 2.0 ** -9 and 2.0 ** -6 in pos and 1.0 in pos and 1.125 in pos
    assert len(np.unique(GRID)) == 253  # 254 finite codes, +0 and -0 coincide


def test_e4m3_round_returns_grid_points_and_the_nearest_one():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=4000) * 3, rng.normal(size=4000) * 200, rng.normal(size=2000) * 0.01,
                        GRID, np.array([0.0, 449.0, 1e9, -1e9, 2.0 ** -10, 2.0 ** -11])])
    r = fp8.e4m3_round(x)
    assert np.all(np.isin(r, GRID))
    clipped = np.clip(x, -448.0, 448.0)
    best = np.min(np.abs(clipped[:, None] - GRID[None, :]), axis=1)
    assert np.allclose(np.abs(r - clipped), best, rtol=0, atol=1e-15)
    assert np.array_equal(fp8.e4m3_round(GRID), GRID)  # grid points are fixed points


def test_ties_go_to_the_even_mantissa():
    # between 1.0 (mantissa 000) and 1.125 (001) -> 1.0; between 1.125 and 1.25 (010) -> 1.25
    assert fp8.e4m3_round(1.0625) == 1.0 and fp8.e4m3_round(1.1875) == 1.25
    # subnormals: step 2^-9; 1.5 steps -> 2 steps (even), 2.5 steps -> 2 steps, 0.5 step -> 0
    assert fp8.e4m3_round(1.5 * 2.0 ** -9) == 2.0 ** -8 and fp8.e4m3_round(2.5 * 2.0 ** -9) == 2.0 ** -8
    assert fp8.e4m3_round(0.5 * 2.0 ** -9) == 0.0
    # top of the range: 464 is the tie between 448 and the missing 480 -> saturates at 448
    assert fp8.e4m3_round(464.0) == 448.0 and fp8.e4m3_round(-1e6) == -448.0


def test_e4m3_round_agrees_with_the_torch_conversion():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.normal(size=20000) * 5, rng.uniform(-440, 440, size=20000),
                        rng.normal(size=5000) * 0.004]).astype(np.float32)
    t = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    assert np.array_equal(fp8.e4m3_round(x.astype(np.float64)), t)


def test_row_and_weight_quantisation():
    rng = np.random.default_rng(2)
    # rows made of grid values times a power of two whose largest magnitude is 448 * 2^j: lossless
    codes = rng.choice(GRID, size=(5, 64))
    codes[:, 0] = 448.0
    j = np.array([-3, 0, 2, -7, 5])
    X = codes * np.exp2(j)[:, None]
    q, s = fp8.quantize_rows(X)
    assert np.array_equal(q, codes) and np.array_equal(s, np.exp2(j))
    # general rows: scale = max|x| / 448 in fp32, error of values in the normal range <= 2^-4 relative
    X = (rng.normal(size=(7, 256)) * 3).astype(np.float32).astype(np.float64)
    q, s = fp8.quantize_rows(X)
    assert np.allclose(s, np.max(np.abs(X), axis=1) / 448.0, rtol=1e-6)
    deq = q * s[:, None]
    big = np.abs(X) > s[:, None] * 2.0 ** -6 * 1.01
    assert np.max(np.abs(deq - X)[big] / np.abs(X)[big]) <= 2.0 ** -4 + 1e-6
    X[0, 5] = s[0] * 2.0 ** -8 * 0.9   # one value in the subnormal range: half a step (2^-10 s) at most
    q, s = fp8.quantize_rows(X)
    assert abs(q[0, 5] * s[0] - X[0, 5]) <= s[0] * 2.0 ** -10 * (1 + 1e-6)
    # weights: gamma folded in before the quantisation
    g = rng.choice([0.5, 1.0, 2.0], size=32)
    Wc = rng.choice(GRID, size=(32, 16)) / g[:, None]
    Wc[0, 0] = 448.0 / g[0]
    wq, sw = fp8.quantize_weights(g, Wc)
    assert sw == 1.0 and np.array_equal(wq, Wc * g[:, None])


@pytest.mark.parametrize("style", [0, 1])
def test_fp8_recompute_reduces_to_the_plain_oracle_on_representable_inputs(style):
    rng = np.random.default_rng(3)
    d_hidden, n_kv, d_head, n = 64, 2, 16, 9
    small = GRID[np.abs(GRID) <= 8.0]
    X = rng.choice(small, size=(n, d_hidden))
    X[:, 0] = 448.0 / 32                      # the largest magnitude of every row: scale 2^-5, codes = 32 x
    W = rng.choice(small, size=(d_hidden, 2 * n_kv * d_head)) / 64.0
    W[0, 0] = 448.0 / 64.0
    gamma = np.ones(d_hidden)
    gk = rng.choice([0.5, 1.0, 1.5], size=d_head)
    pos = rng.integers(0, 500, size=n)
    Kp, Vp = oracle.recompute_kv(X, pos, gamma, W, n_kv, d_head, 1e-6, 1e4, gk, 1e-6, style)
    Kq, Vq = fp8.recompute_kv_fp8(X, pos, gamma, W, n_kv, d_head, 1e-6, 1e4, gk, 1e-6, style)
    assert np.allclose(Kq, Kp, rtol=1e-12, atol=1e-12) and np.allclose(Vq, Vp, rtol=1e-12, atol=1e-12)


def test_fp8_recompute_stays_within_the_formats_error_of_the_plain_oracle():
    rng = np.random.default_rng(4)
    d_hidden, n_kv, d_head, n = 512, 2, 64, 40
    X = (rng.normal(size=(n, d_hidden))).astype(np.float32).astype(np.float64)
    W = (rng.normal(size=(d_hidden, 2 * n_kv * d_head)) * 0.02).astype(np.float32).astype(np.float64)
    gamma = np.ones(d_hidden)
    pos = np.arange(n)
    Kp, Vp = oracle.recompute_kv(X, pos, gamma, W, n_kv, d_head, 1e-6, 1e4, None, 0.0, 0)
    Kq, Vq = fp8.recompute_kv_fp8(X, pos, gamma, W, n_kv, d_head, 1e-6, 1e4, None, 0.0, 0)
    # two operands with <= 2^-4 relative error each, errors independent over 512 terms: a few percent of the
    # output's rms, and nowhere near 2 * 2^-4 of it
    for a, b in ((Kq, Kp), (Vq, Vp)):
        rel = np.linalg.norm(a - b) / np.linalg.norm(b)
        assert 0.005 < rel < 0.08, rel
