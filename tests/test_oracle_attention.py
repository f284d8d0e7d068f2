"""Pins for the oracle's decode attention (Eq. 6-7) -- no GPU.

Hand cases, degenerate cases with a known answer, invariances (permutation, position shift through
the rotation, split/merge by log-sum-exp), the grouped-head mapping, the window mask, and a
brute-force pure-Python evaluation on tiny inputs.
"""
import math

import numpy as np
import pytest

import oracle


def _brute(q, q_pos, K, V, kpos, scale, window, group):
    """Eq. 6-7 with Python scalars only."""
    n_q, d = len(q), len(q[0])
    out = [[0.0] * d for _ in range(n_q)]
    for h in range(n_q):
        g = h // group
        scores = []
        for j in range(len(K)):
            dlt = q_pos - kpos[j]
            if dlt < 0 or (window and dlt >= window):
                continue
            scores.append((j, scale * sum(q[h][c] * K[j][g][c] for c in range(d))))
        m = max(s for _, s in scores)
        den = sum(math.exp(s - m) for _, s in scores)
        for j, s in scores:
            p = math.exp(s - m) / den
            for c in range(d):
                out[h][c] += p * V[j][g][c]
    return np.array(out)


def test_hand_case_two_keys():
    # d_head = 2, one head, scale = 1: scores (0, ln 3) -> weights (1/4, 3/4)
    q = np.array([[1.0, 0.0]])
    K = np.array([[[0.0, 5.0]], [[math.log(3.0), -2.0]]])
    V = np.array([[[4.0, 0.0]], [[0.0, 8.0]]])
    out = oracle.decode_attention(q, 1, [(K, V, 0)], 1.0)
    np.testing.assert_allclose(out, [[1.0, 6.0]], rtol=1e-14)
    # the 1/sqrt(d_head) scale of Eq. 6 enters inside the softmax
    out = oracle.decode_attention(q * math.sqrt(2.0), 1, [(K, V, 0)], 1.0 / math.sqrt(2.0))
    np.testing.assert_allclose(out, [[1.0, 6.0]], rtol=1e-14)


def test_single_key_returns_value_and_equal_keys_average():
    rng = np.random.default_rng(0)
    q = rng.standard_normal((4, 8))
    K = rng.standard_normal((1, 2, 8))
    V = rng.standard_normal((1, 2, 8))
    out = oracle.decode_attention(q, 0, [(K, V, 0)], 0.3)
    np.testing.assert_allclose(out[0], V[0, 0], rtol=1e-15)
    np.testing.assert_allclose(out[3], V[0, 1], rtol=1e-15)
    K5 = np.repeat(K, 5, axis=0)
    V5 = rng.standard_normal((5, 2, 8))
    out = oracle.decode_attention(q, 4, [(K5, V5, 0)], 0.3)
    np.testing.assert_allclose(out[1], V5[:, 0].mean(axis=0), rtol=1e-13)
    np.testing.assert_allclose(out[2], V5[:, 1].mean(axis=0), rtol=1e-13)


def test_grouped_heads_map_consecutively_and_mha_is_the_special_case():
    rng = np.random.default_rng(1)
    n_q, n_kv, d = 6, 3, 4
    q = rng.standard_normal((n_q, d))
    K = rng.standard_normal((7, n_kv, d))
    V = rng.standard_normal((7, n_kv, d))
    out = oracle.decode_attention(q, 6, [(K, V, 0)], 0.5)
    # expand K/V so that every query head has its own KV head (MHA) with g = h // 2
    Kx = np.repeat(K, 2, axis=1)
    Vx = np.repeat(V, 2, axis=1)
    out_mha = oracle.decode_attention(q, 6, [(Kx, Vx, 0)], 0.5)
    assert np.array_equal(out, out_mha)
    ref = _brute(q.tolist(), 6, K.tolist(), V.tolist(), list(range(7)), 0.5, 0, 2)
    np.testing.assert_allclose(out, ref, rtol=1e-13)


def test_brute_force_with_window_and_future_keys():
    rng = np.random.default_rng(2)
    q = rng.standard_normal((2, 4))
    K = rng.standard_normal((12, 1, 4))
    V = rng.standard_normal((12, 1, 4))
    # keys at positions 3..14; query at 10 with window 4 sees positions 7, 8, 9, 10 only
    out = oracle.decode_attention(q, 10, [(K, V, 3)], 0.7, window=4)
    ref = _brute(q.tolist(), 10, K.tolist(), V.tolist(), list(range(3, 15)), 0.7, 4, 2)
    np.testing.assert_allclose(out, ref, rtol=1e-13)
    sel = slice(7 - 3, 10 - 3 + 1)
    out_sel = oracle.decode_attention(q, 10, [(K[sel], V[sel], 7)], 0.7, window=0)
    np.testing.assert_allclose(out, out_sel, rtol=1e-13)
    # window = 1 sees only the query's own position
    out1 = oracle.decode_attention(q, 10, [(K, V, 3)], 0.7, window=1)
    np.testing.assert_allclose(out1[0], V[7, 0], rtol=1e-15)


def test_permutation_invariance():
    rng = np.random.default_rng(3)
    q = rng.standard_normal((2, 8))
    K = rng.standard_normal((9, 2, 8))
    V = rng.standard_normal((9, 2, 8))
    perm = rng.permutation(9)
    a = oracle.decode_attention(q, 8, [(K, V, 0)], 0.35)
    b = oracle.decode_attention(q, 8, [(K[perm], V[perm], 0)], 0.35)
    np.testing.assert_allclose(a, b, rtol=1e-12)


def test_segments_equal_concatenation_and_lse_merge():
    # Algorithm 1's CONCAT(old, window, current): the result over three segments equals the result
    # over the concatenated cache, and equals the log-sum-exp merge of per-segment partial results.
    rng = np.random.default_rng(4)
    n_q, n_kv, d = 4, 2, 16
    q = rng.standard_normal((n_q, d))
    K = rng.standard_normal((20, n_kv, d))
    V = rng.standard_normal((20, n_kv, d))
    scale = 0.25
    whole = oracle.decode_attention(q, 19, [(K, V, 0)], scale)
    cuts = [(0, 12), (12, 19), (19, 20)]
    segs = [(K[a:b], V[a:b], a) for a, b in cuts]
    assert np.array_equal(oracle.decode_attention(q, 19, segs, scale), whole)
    # merge partials: o = sum_s w_s o_s, w_s = exp(lse_s) / sum exp(lse)
    parts, lses = [], []
    for a, b in cuts:
        parts.append(oracle.decode_attention(q, 19, [(K[a:b], V[a:b], a)], scale))
        s = scale * np.einsum("hc,jhc->hj", q, np.repeat(K[a:b], n_q // n_kv, axis=1))
        lses.append(np.log(np.exp(s).sum(axis=1)))
    lses = np.array(lses)
    wts = np.exp(lses - lses.max(axis=0))
    wts /= wts.sum(axis=0)
    merged = sum(wts[i][:, None] * parts[i] for i in range(3))
    np.testing.assert_allclose(merged, whole, rtol=1e-12)


@pytest.mark.parametrize("style", [oracle.ROPE_INTERLEAVED, oracle.ROPE_HALF])
def test_shifting_all_positions_leaves_attention_unchanged(style):
    # <R_p q, R_j k> = <R_{p-j} q, k>: rotate q and k at positions shifted by a constant and the
    # output must not move (also the reason absolute and window-relative positions agree when q
    # and k share the convention).
    rng = np.random.default_rng(5)
    d, theta = 32, 1.0e4
    q0 = rng.standard_normal((2, d))
    k0 = rng.standard_normal((6, 1, d))
    V = rng.standard_normal((6, 1, d))
    outs = []
    for shift in (0, 17, 1000):
        q = np.stack([oracle.rope(q0[h], 5 + shift, theta, style) for h in range(2)])
        K = np.stack([oracle.rope(k0[j, 0], j + shift, theta, style) for j in range(6)])[:, None, :]
        outs.append(oracle.decode_attention(q, 5 + shift, [(K, V, shift)], 1.0 / math.sqrt(d)))
    np.testing.assert_allclose(outs[1], outs[0], rtol=1e-10)
    np.testing.assert_allclose(outs[2], outs[0], rtol=1e-9)


def test_rope_styles_give_the_same_scores():
    # the two pairings differ by one channel permutation applied to q and k alike
    rng = np.random.default_rng(6)
    d, theta = 16, 1.0e4
    perm = np.concatenate([np.arange(0, d, 2), np.arange(1, d, 2)])
    q0 = rng.standard_normal(d)
    k0 = rng.standard_normal((5, d))
    V = rng.standard_normal((5, 1, d))
    q_i = oracle.rope(q0, 4, theta, oracle.ROPE_INTERLEAVED)[None]
    K_i = np.stack([oracle.rope(k0[j], j, theta, oracle.ROPE_INTERLEAVED) for j in range(5)])[:, None]
    q_h = oracle.rope(q0[perm], 4, theta, oracle.ROPE_HALF)[None]
    K_h = np.stack([oracle.rope(k0[j][perm], j, theta, oracle.ROPE_HALF) for j in range(5)])[:, None]
    a = oracle.decode_attention(q_i, 4, [(K_i, V, 0)], 0.25)
    b = oracle.decode_attention(q_h, 4, [(K_h, V, 0)], 0.25)
    np.testing.assert_allclose(a, b, rtol=1e-12)


def test_softmax_is_shift_stable():
    # large scores must not overflow: result equals the one with all scores reduced by a constant
    q = np.array([[1.0, 0.0]])
    K = np.array([[[800.0, 0.0]], [[800.0 + math.log(3.0), 0.0]]])
    V = np.array([[[4.0, 0.0]], [[0.0, 8.0]]])
    out = oracle.decode_attention(q, 1, [(K, V, 0)], 1.0)
    np.testing.assert_allclose(out, [[1.0, 6.0]], rtol=1e-12)
