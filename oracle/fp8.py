"""Oracle for the FP8 checkpoint variant (test infrastructure only; never imported by the product path).

The paper names lower-precision checkpoints as future work (its Section 6, second item) and fixes no
format, so the variant is defined here and in include/kvd.h:

  * a residual row x (bf16) is stored as E4M3 codes with one fp32 scale per row,
        s_x = max(|x|) / 448,   code_k = e4m3_rne_sat(x_k * r_x),  r_x = 448 / max(|x|)   (all in fp32),
    together with the row's sum of squares taken from the ORIGINAL row (the RMSNorm statistic of Eq. 2 is
    not affected by the quantisation);
  * the folded weights W' = gamma (.) W_kv (Eq. 1 composed with Eq. 13-14) are stored as E4M3 codes with one
    fp32 scale for the whole matrix, s_w = max|W'| / 448, code = e4m3_rne_sat(W' * (448 / max|W'|)), W' and
    the reciprocal formed in fp32 (a multiplication by the rounded reciprocal, not a division: one division
    per row instead of one per element on the GPU; the decoded value is still code * s);
  * RECOMPUTE_KV then is Eq. 13-14 on the dequantised operands:
        y = (s_x s_w / rms(x)) * sum_k code_x[k] code_w[k][:]      followed by key norm and rotation as usual.

`e4m3_round` is written from the format's definition (1 sign, 4 exponent bits with bias 7, 3 mantissa bits,
no infinities, largest finite value 448, subnormal step 2^-9, round to nearest even, saturating); its pins
(tests/test_oracle_fp8.py) are the value table implied by that definition, hand-picked ties, and PyTorch's
own float8_e4m3fn conversion on the CPU as an independent library routine.

The codes are an encoding decided in floating point, so the definition fixes the precision of that
decision: the scale, the reciprocal, the product and the rounding input are fp32.  The definition is
frozen: a change to this file's arithmetic has to name the reading of the paper that calls for it, never a
property of an implementation.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np

E4M3_MAX = 448.0


def e4m3_round(x) -> np.ndarray:
    """Nearest E4M3 value (ties to even, saturating at +-448) of every element; result in fp64."""
    x = np.asarray(x, dtype=np.float64)
    a = np.minimum(np.abs(x), E4M3_MAX)
    # exponent of the binade: values in [2^e, 2^(e+1)) have spacing 2^(e-3); below 2^-6 the spacing is 2^-9
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.maximum(e, -6.0)
    step = np.exp2(e - 3.0)
    q = np.rint(a / step) * step          # np.rint rounds half to even; a / step is exact (power of two)
    q = np.minimum(q, E4M3_MAX)
    return np.copysign(q, x)


def quantize_rows(X_f64: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Per-row quantisation of bf16-valued rows.  Returns (values on the E4M3 grid as fp64 [n, d], scales
    fp64 [n]) with row r represented by values[r] * scales[r].  Scale and quotient are formed in fp32."""
    X = np.asarray(X_f64, dtype=np.float32)
    amax = np.max(np.abs(X), axis=1)
    amax = np.maximum(amax, np.float32(1e-30))
    s = (amax / np.float32(E4M3_MAX)).astype(np.float32)
    r = (np.float32(E4M3_MAX) / amax).astype(np.float32)
    quot = (X * r[:, None]).astype(np.float32)
    return e4m3_round(quot.astype(np.float64)), s.astype(np.float64)


def quantize_weights(gamma_f64: np.ndarray, W_f64: np.ndarray) -> Tuple[np.ndarray, float]:
    """W' = gamma (.) W formed in fp32 (exact for bf16 inputs), one scale for the matrix.  Returns (values on
    the E4M3 grid [d_hidden, n_cols] as fp64, scale)."""
    Wp = (np.asarray(gamma_f64, dtype=np.float32)[:, None] * np.asarray(W_f64, dtype=np.float32)).astype(np.float32)
    amax = np.float32(np.max(np.abs(Wp)))
    amax = np.float32(max(amax, np.float32(1e-30)))
    s = amax / np.float32(E4M3_MAX)
    quot = (Wp * (np.float32(E4M3_MAX) / amax)).astype(np.float32)
    return e4m3_round(quot.astype(np.float64)), float(s)


def recompute_kv_fp8(X, pos, gamma_in, W_kv, n_kv: int, d_head: int, rms_eps: float, theta: float,
                     gamma_k=None, qk_eps: float = 0.0, rope_style: int = 0):
    """Eq. 13-14 from FP8 checkpoints as defined above: (K, V) in fp64, each [n, n_kv, d_head].

    The linear part is written out here (the statistic comes from the original row, which the plain
    oracle's fused norm cannot express); key norm and rotation follow the plain oracle's definitions."""
    X = np.asarray(X, dtype=np.float64)
    xq, sx = quantize_rows(X)
    wq, sw = quantize_weights(gamma_in, W_kv)
    rstd = 1.0 / np.sqrt(np.mean(X * X, axis=1) + rms_eps)   # Eq. 2 on the ORIGINAL row
    Y = ((xq * sx[:, None]) * rstd[:, None]) @ (wq * sw)     # [n, 2 * n_kv * d_head]
    return _finish_heads(Y, pos, n_kv, d_head, theta, gamma_k, qk_eps, rope_style)


def _finish_heads(Y: np.ndarray, pos, n_kv: int, d_head: int, theta: float, gamma_k, qk_eps: float, rope_style: int):
    """Key norm over d_head (when gamma_k is given), rotation of the keys by their positions (Eq. 11-12 via the
    plain oracle's rope), values unchanged."""
    import oracle
    n = Y.shape[0]
    kdim = n_kv * d_head
    K = Y[:, :kdim].reshape(n, n_kv, d_head).copy()
    V = Y[:, kdim:].reshape(n, n_kv, d_head).copy()
    if gamma_k is not None:
        gk = np.asarray(gamma_k, dtype=np.float64)
        K = K / np.sqrt(np.mean(K * K, axis=2, keepdims=True) + qk_eps) * gk[None, None, :]
    for r in range(n):
        for h in range(n_kv):
            K[r, h] = oracle.rope(K[r, h], int(pos[r]), theta, rope_style)
    return K, V
