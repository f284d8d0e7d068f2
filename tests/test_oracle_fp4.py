"""Pins of the FP4-checkpoint oracle (CPU only).

  * e2m1_round against the value table that the format's definition implies (all 16 codes decoded from their bit
    fields), brute-force nearest over that table, and hand-computed ties;
  * quantize_rows_fp4: the row scale is the stated power of two, block scales lie on the E4M3 grid, exactly
    representable rows survive unchanged, every element is within one block-scale unit of its original (half a
    step of the coarsest binade), decoded values are exact in bf16;
  * recompute_kv_fp4 reduces to the plain (already pinned) oracle when the rows are exactly representable and
    stays within the format's error of it otherwise.
"""
import numpy as np

import oracle
from oracle import fp4, fp8
from kvd_synth import GEMMA3_4B_GLOBAL, TINY_GQA, bf16_to_f64, f32_to_bf16_bits, make_layer_weights, make_residuals


def decode_e2m1(code: int) -> float:
    """Value of an E2M1 code from its fields: sign(1) exponent(2, bias 1) mantissa(1); no infinities, no NaNs."""
    s = -1.0 if code & 0x8 else 1.0
    e, m = (code >> 1) & 0x3, code & 1
    if e == 0:
        return s * m * 0.5
    return s * (1 + m / 2.0) * 2.0 ** (e - 1)


GRID = np.array(sorted({decode_e2m1(c) for c in range(16)}))


def test_the_grid_is_the_formats():
    assert GRID.tolist() == [-6.0, -4.0, -3.0, -2.0, -1.5, -1.0, -0.5, 0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def test_e2m1_round_returns_the_nearest_grid_point():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=5000) * 2.5, rng.uniform(-7, 7, size=5000), GRID, [0.0, 6.1, 100.0, -100.0, 1e-9]])
    r = fp4.e2m1_round(x)
    assert np.all(np.isin(r, GRID))
    clipped = np.clip(x, -6.0, 6.0)
    best = np.min(np.abs(clipped[:, None] - GRID[None, :]), axis=1)
    assert np.allclose(np.abs(r - clipped), best, rtol=0, atol=1e-15)
    assert np.array_equal(fp4.e2m1_round(GRID), GRID)


def test_ties_go_to_the_even_code():
    # codes: 0 -> 0, 1 -> 0.5, 2 -> 1, 3 -> 1.5, 4 -> 2, 5 -> 3, 6 -> 4, 7 -> 6
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    for x, want in ties.items():
        assert fp4.e2m1_round(x) == want, x
        assert fp4.e2m1_round(-x) == -want, x
    assert fp4.e2m1_round(7.0) == 6.0 and fp4.e2m1_round(-1e9) == -6.0
    assert fp4.e2m1_round(np.nextafter(0.25, 1.0)) == 0.5 and fp4.e2m1_round(np.nextafter(5.0, 6.0)) == 6.0


def test_quantisation_structure_and_error_bound():
    X = bf16_to_f64(make_residuals(GEMMA3_4B_GLOBAL, 64, seed=3, outliers=True))
    X[5] = 0.0                     # an all-zero row
    X[6, 32:48] = 0.0              # an all-zero block
    codes, block, row = fp4.quantize_rows_fp4(X)
    amax = np.max(np.abs(X), axis=1)
    nz = amax > 0
    assert np.all(np.log2(row) == np.round(np.log2(row)))                 # powers of two
    assert np.all((amax[nz] / row[nz] >= 1024) & (amax[nz] / row[nz] < 2048))
    assert row[5] == 1.0 and np.all(codes[5] == 0)
    assert np.array_equal(fp8.e4m3_round(block), block)                   # on the E4M3 grid
    assert np.all(np.isin(np.abs(codes), GRID[GRID >= 0]))
    assert np.all(codes[6, 32:48] == 0)
    xhat = fp4.dequantize_rows_fp4(codes, block, row)
    # exact in bf16
    assert np.array_equal(bf16_to_f64(f32_to_bf16_bits(xhat.astype(np.float32))), xhat)
    # every element within one unit of its block's decode scale (half the coarsest step, or the saturation gap)
    d = np.repeat(block * row[:, None], 16, axis=1)
    assert np.all(np.abs(X - xhat) <= d * (1 + 1e-6))
    # the largest element of a block decodes to within 1/16 of itself (the block scale's three mantissa bits)
    Xb, Hb = np.abs(X).reshape(64, -1, 16), np.abs(xhat).reshape(64, -1, 16)
    i = np.argmax(Xb, axis=2)[..., None]
    top, top_hat = np.take_along_axis(Xb, i, 2)[..., 0], np.take_along_axis(Hb, i, 2)[..., 0]
    ok = top > 0
    assert np.all(np.abs(top_hat[ok] - top[ok]) <= top[ok] / 8)
    rel = np.linalg.norm(X - xhat) / np.linalg.norm(X)
    assert 0.02 < rel < 0.25, rel   # the format's accuracy on rows with outlier channels: reported, not claimed


def _representable_rows(n, d, seed):
    """Rows made of E2M1 grid values times per-block powers of two, every block containing a +-6 entry: the
    quantiser must reproduce them exactly."""
    rng = np.random.default_rng(seed)
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6])
    vals = rng.choice(grid, size=(n, d // 16, 16)) * rng.choice([-1.0, 1.0], size=(n, d // 16, 16))
    vals[:, :, 0] = 6.0 * rng.choice([-1.0, 1.0], size=(n, d // 16))
    j = rng.integers(-5, 3, size=(n, d // 16))  # block magnitudes within 2^8 of each other: scales stay normal E4M3
    j[:, 0] = 2                                  # the row's largest block
    return (vals * np.exp2(j)[:, :, None]).reshape(n, d)


def test_representable_rows_survive_and_the_recompute_reduces_to_the_plain_oracle():
    shape = TINY_GQA
    w = make_layer_weights(shape)
    X = _representable_rows(24, shape.d_hidden, 1)
    assert np.array_equal(bf16_to_f64(f32_to_bf16_bits(X.astype(np.float32))), X)
    codes, block, row = fp4.quantize_rows_fp4(X)
    assert np.array_equal(fp4.dequantize_rows_fp4(codes, block, row), X)
    pos = np.arange(24) + 3
    args = (bf16_to_f64(w.gamma_in), bf16_to_f64(w.w_kv), shape.n_kv_heads, shape.d_head, shape.rms_eps, shape.rope_theta,
            bf16_to_f64(w.gamma_k), shape.rms_eps)
    K4, V4 = fp4.recompute_kv_fp4(X, pos, *args)
    K, V = oracle.recompute_kv(X, pos, *args)
    assert np.allclose(K4, K, rtol=1e-11, atol=1e-12) and np.allclose(V4, V, rtol=1e-11, atol=1e-12)


def test_recompute_from_fp4_rows_stays_within_the_formats_error():
    shape = TINY_GQA
    w = make_layer_weights(shape)
    X = bf16_to_f64(make_residuals(shape, 48, seed=4))
    pos = np.arange(48)
    args = (bf16_to_f64(w.gamma_in), bf16_to_f64(w.w_kv), shape.n_kv_heads, shape.d_head, shape.rms_eps, shape.rope_theta,
            bf16_to_f64(w.gamma_k), shape.rms_eps)
    K4, V4 = fp4.recompute_kv_fp4(X, pos, *args)
    K, V = oracle.recompute_kv(X, pos, *args)
    # V is linear in the row: its error is the row error seen through W; relative to V it stays near the row's
    xhat = fp4.dequantize_rows_fp4(*fp4.quantize_rows_fp4(X))
    row_rel = np.linalg.norm(X - xhat) / np.linalg.norm(X)
    v_rel = np.linalg.norm(V4 - V) / np.linalg.norm(V)
    assert 0.3 * row_rel < v_rel < 3 * row_rel, (row_rel, v_rel)
    assert np.linalg.norm(K4 - K) / np.linalg.norm(K) < 3 * row_rel
