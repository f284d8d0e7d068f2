"""Oracle for the FP4 checkpoint variant (test infrastructure only; never imported by the product path).

The paper names lower-precision checkpoints as future work (its Section 6, second item) and fixes no format.
This variant stores a residual row in 4-bit codes with two levels of scales -- the layout NVIDIA calls NVFP4
(E2M1 codes, one E4M3 scale per block of 16 channels, one more scale per tensor), with the outer scale taken
per row and restricted to a power of two so that decoding is exact in bf16.  Defined here and in include/kvd.h:

  * row scale       s_row = 2^(E - 10), E = floor(log2(max|x|))          (1 when the row is all zeros), so that
                    max|x| / s_row lies in [1024, 2048);
  * block scale     for every block of 16 consecutive channels: t = (max|x_block| / 6) / s_row, formed in fp32
                    (the division by 6 rounds, the division by s_row is exact), b = e4m3(t) rounded to nearest
                    even (t <= 341.4 < 448: never saturates); the block decodes with d = b * s_row (exact);
  * codes           c = e2m1(x / d), the quotient formed in fp32, rounded to the nearest of
                    {0, 0.5, 1, 1.5, 2, 3, 4, 6} (ties to the even code, saturating at 6); a block whose scale
                    rounds to zero has all codes zero;
  * decoded value   x^ = c * d, exact in bf16 (two significant bits times four times a power of two);
  * the row's sum of squares is taken from the ORIGINAL row (the RMSNorm statistic of Eq. 2 is not affected by
    the quantisation), as in the FP8 variant.
RECOMPUTE_KV from such rows is Eq. 13-14 on x^ with 1/rms of the original row: the rows are expanded back to bf16
and go through the ordinary projection (the weights stay bf16).  Per token and layer the store holds
d_hidden/2 + d_hidden/16 + 12 bytes (1,452 for d_hidden = 2560 against 5,128 for bf16 rows and 4,096 for the K/V
they replace).

`e2m1_round` is written from the format's definition (1 sign, 2 exponent bits with bias 1, 1 mantissa bit; no
infinities or NaNs; subnormal step 0.5; largest value 6).  Pins: tests/test_oracle_fp4.py (the value table from the
bit fields, brute-force nearest, hand-picked ties, exactly representable rows, the error bound, reduction to the
plain oracle).  The definition is frozen: a change to this file's arithmetic has to name the reading of the paper
that calls for it, never a property of an implementation.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np

from .fp8 import _finish_heads, e4m3_round

E2M1_MAX = 6.0
BLOCK = 16


def e2m1_round(x) -> np.ndarray:
    """Nearest E2M1 value (ties to the even code, saturating at +-6) of every element; result in fp64."""
    x = np.asarray(x, dtype=np.float64)
    a = np.abs(x)
    # binade [2^e, 2^(e+1)) has spacing 2^(e-1) for e = 0, 1, 2; below 1 the spacing is 0.5 (the subnormal step)
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.clip(e, 0.0, 2.0)
    step = np.exp2(e - 1.0)
    q = np.rint(a / step) * step  # np.rint rounds half to even; even multiples of the step are the even codes
    q = np.minimum(q, E2M1_MAX)
    return np.copysign(q, x)


def quantize_rows_fp4(X_f64: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Rows [n, d] (bf16-valued, d a multiple of 16) -> (code values on the E2M1 grid [n, d], block scales on the
    E4M3 grid [n, d/16], row scales [n], all fp64).  Element (r, k) decodes as codes[r, k] * block[r, k // 16] * row[r].
    Every floating-point decision is taken in fp32, as the definition states."""
    X = np.asarray(X_f64, dtype=np.float32)
    n, d = X.shape
    assert d % BLOCK == 0
    amax = np.max(np.abs(X), axis=1)
    _, ex = np.frexp(amax)  # amax = m * 2^ex with m in [0.5, 1): floor(log2(amax)) = ex - 1
    s_row = np.where(amax > 0, np.exp2((ex - 1 - 10).astype(np.float64)), 1.0).astype(np.float32)
    Xb = X.reshape(n, d // BLOCK, BLOCK)
    bmax = np.max(np.abs(Xb), axis=2)
    t = ((bmax / np.float32(6.0)).astype(np.float32) / s_row[:, None]).astype(np.float32)
    assert np.all(t <= 448.0)
    b = e4m3_round(t.astype(np.float64))
    dscale = (b.astype(np.float32) * s_row[:, None]).astype(np.float32)  # exact
    with np.errstate(divide="ignore", invalid="ignore"):
        quot = np.where(dscale[:, :, None] > 0, (Xb / dscale[:, :, None]).astype(np.float32), np.float32(0.0))
    codes = e2m1_round(quot.astype(np.float64)).reshape(n, d)
    return codes, b, s_row.astype(np.float64)


def dequantize_rows_fp4(codes: np.ndarray, block: np.ndarray, row: np.ndarray) -> np.ndarray:
    """The decoded rows x^ [n, d] in fp64 (exactly representable in bf16)."""
    n, d = codes.shape
    return (codes.reshape(n, d // BLOCK, BLOCK) * (block * row[:, None])[:, :, None]).reshape(n, d)


def recompute_kv_fp4(X, pos, gamma_in, W_kv, n_kv: int, d_head: int, rms_eps: float, theta: float,
                     gamma_k=None, qk_eps: float = 0.0, rope_style: int = 0):
    """Eq. 13-14 from FP4 checkpoints as defined above: (K, V) in fp64, each [n, n_kv, d_head].  The linear part
    is written out here (the statistic comes from the original row); key norm and rotation follow the plain
    oracle's definitions."""
    X = np.asarray(X, dtype=np.float64)
    xhat = dequantize_rows_fp4(*quantize_rows_fp4(X))
    rstd = 1.0 / np.sqrt(np.mean(X * X, axis=1) + rms_eps)  # Eq. 2 on the ORIGINAL row
    Y = (xhat * rstd[:, None] * np.asarray(gamma_in, dtype=np.float64)[None, :]) @ np.asarray(W_kv, dtype=np.float64)
    return _finish_heads(Y, pos, n_kv, d_head, theta, gamma_k, qk_eps, rope_style)
