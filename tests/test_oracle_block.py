"""Pins for ``oracle.stack.OracleStack._block`` and the logits (Eq. 3-9, Algorithm 1) -- no GPU.

Every intermediate of a tiny decoder stack is worked out here with Python scalars and lists, straight
from the equations, without calling anything under ``oracle``: RMSNorm (Eq. 1-2), the query / key /
value projections (Eq. 3-5), the per-head query and key norms, the rotation of consecutive channel
pairs (Eq. 11-12), the softmax over the keys seen so far (Eq. 6-7), the output projection and the
residual add (Eq. 8), the gated MLP and its residual add (Eq. 9), the final norm, the vocabulary
projection and the greedy pick.  The oracle's logits must agree to rounding.

The second half shows that the pin has teeth: the same hand computation is compared with the oracle
run on deliberately wrong weights or shapes (W_o dropped, gate and up exchanged, the other activation,
another query-head -> KV-head grouping, key norm scale left out, no rotation) and must then DISAGREE.
"""
import math
from dataclasses import replace

import numpy as np
import pytest

from kvd_synth import ROPE_HALF, ROPE_INTERLEAVED, StackShape
from oracle.stack import OracleStack

EPS = 1e-3  # large enough to matter in the hand computation


def _mat(rows, cols, salt):
    """A small deterministic matrix without symmetry: entries in [-0.6, 0.6], no two rows alike."""
    return [[((7 * i + 3 * j + salt * 5 + (i * j) % 4) % 13 - 6) / 10.0 for j in range(cols)] for i in range(rows)]


def _vec(n, salt):
    """Norm scales that are clearly not 1."""
    return [0.7 + 0.15 * ((i + salt) % 5) for i in range(n)]


def _tiny(activation="gelu_tanh", n_layers=1, style=ROPE_INTERLEAVED, qk_norm=True):
    # 4 query heads on 2 KV heads (groups of two), d_head 4 (two rotation pairs with different
    # frequencies), d_hidden 3, MLP width 5, vocabulary 3
    return StackShape("hand", n_layers, 3, 4, 2, 4, 5, 3, EPS, qk_norm, 50.0, 50.0, 0, 0, activation, style)


def _weights(s):
    nq, nkv, dh, d = s.n_q_heads, s.n_kv_heads, s.d_head, s.d_hidden
    layers = []
    for l in range(s.n_layers):
        layers.append({
            "w_q": _mat(d, nq * dh, 1 + 10 * l), "w_kv": _mat(d, 2 * nkv * dh, 2 + 10 * l),
            "w_o": _mat(nq * dh, d, 3 + 10 * l), "w_gate": _mat(d, s.d_mlp, 4 + 10 * l),
            "w_up": _mat(d, s.d_mlp, 5 + 10 * l), "w_down": _mat(s.d_mlp, d, 6 + 10 * l),
            "gamma_in": _vec(d, 0 + l), "gamma_mlp": _vec(d, 1 + l), "gamma_q": _vec(dh, 2 + l),
            "gamma_k": _vec(dh, 3 + l),
        })
    return {"embed": _mat(s.vocab, d, 7), "lm_head": _mat(d, s.vocab, 8), "gamma_final": _vec(d, 4),
            "layers": layers}


def _as_arrays(w):
    out = {k: np.asarray(v, dtype=np.float64) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: np.asarray(v, dtype=np.float64) for k, v in lw.items()} for lw in w["layers"]]
    return out


# ------------------------------------------------------------------ the equations, with scalars
def _rmsnorm(x, gamma, eps):
    r = math.sqrt(sum(v * v for v in x) / len(x) + eps)  # Eq. 2 (+ eps inside the root)
    return [v / r * g for v, g in zip(x, gamma)]  # Eq. 1


def _vecmat(x, w):
    return [sum(x[i] * w[i][c] for i in range(len(x))) for c in range(len(w[0]))]


def _rotate(x, pos, theta, style):
    dh = len(x)
    y = list(x)
    for i in range(dh // 2):  # Eq. 11-12: pair i turns by pos * theta^(-2i/d_head)
        phi = pos * theta ** (-2.0 * i / dh)
        ia, ib = (i, i + dh // 2) if style == ROPE_HALF else (2 * i, 2 * i + 1)
        y[ia] = x[ia] * math.cos(phi) - x[ib] * math.sin(phi)
        y[ib] = x[ia] * math.sin(phi) + x[ib] * math.cos(phi)
    return y


def _gelu_tanh(v):
    return 0.5 * v * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (v + 0.044715 * v ** 3)))


def _silu(v):
    return v / (1.0 + math.exp(-v))


def _hand_logits(s, w, tokens, first_step_shortcut=False):
    """Algorithm 1 with an unbounded cache, token by token; returns the logits of every step."""
    nq, nkv, dh = s.n_q_heads, s.n_kv_heads, s.d_head
    act = _gelu_tanh if s.activation == "gelu_tanh" else _silu
    cache = [[] for _ in range(s.n_layers)]  # per layer: list of (K_j [nkv][dh], V_j [nkv][dh])
    all_logits = []
    for pos, tok in enumerate(tokens):
        h = list(w["embed"][tok])
        for l in range(s.n_layers):
            lw = w["layers"][l]
            xb = _rmsnorm(h, lw["gamma_in"], s.rms_eps)
            q = _vecmat(xb, lw["w_q"])  # Eq. 3
            kv = _vecmat(xb, lw["w_kv"])  # Eq. 4-5, K columns first
            qh = [q[a * dh:(a + 1) * dh] for a in range(nq)]
            kh = [kv[g * dh:(g + 1) * dh] for g in range(nkv)]
            vh = [kv[nkv * dh + g * dh: nkv * dh + (g + 1) * dh] for g in range(nkv)]
            if s.qk_norm:
                qh = [_rmsnorm(x, lw["gamma_q"], s.rms_eps) for x in qh]
                kh = [_rmsnorm(x, lw["gamma_k"], s.rms_eps) for x in kh]
            qh = [_rotate(x, pos, s.theta_global, s.rope_style) for x in qh]
            kh = [_rotate(x, pos, s.theta_global, s.rope_style) for x in kh]
            cache[l].append((kh, vh))
            heads = []
            for a in range(nq):
                g = a // (nq // nkv)  # consecutive query heads share a KV head
                if first_step_shortcut and pos == 0:
                    heads += vh[g]  # a softmax over one key is 1: the head's output is V_t itself
                    continue
                sc = [sum(qh[a][c] * kj[g][c] for c in range(dh)) / math.sqrt(dh) for kj, _ in cache[l]]  # Eq. 6
                m = max(sc)
                p = [math.exp(v - m) for v in sc]
                z = sum(p)
                heads += [sum(p[j] * cache[l][j][1][g][c] for j in range(len(p))) / z for c in range(dh)]  # Eq. 7
            att = _vecmat(heads, lw["w_o"])
            h = [a + b for a, b in zip(h, att)]  # Eq. 8
            xm = _rmsnorm(h, lw["gamma_mlp"], s.rms_eps)
            gate, up = _vecmat(xm, lw["w_gate"]), _vecmat(xm, lw["w_up"])
            mlp = _vecmat([act(a) * b for a, b in zip(gate, up)], lw["w_down"])
            h = [a + b for a, b in zip(h, mlp)]  # Eq. 9
        all_logits.append(_vecmat(_rmsnorm(h, w["gamma_final"], s.rms_eps), w["lm_head"]))
    return all_logits


def _oracle_logits(s, w, tokens, policy="full", budget=0):
    m = OracleStack(s, _as_arrays(w), policy, budget)
    return [m.step(t) for t in tokens]


TOKENS = [2, 0, 1]


# ------------------------------------------------------------------ the pins
@pytest.mark.parametrize("activation", ["gelu_tanh", "silu"])
@pytest.mark.parametrize("style", [ROPE_INTERLEAVED, ROPE_HALF])
@pytest.mark.parametrize("n_layers", [1, 2])
def test_block_and_logits_match_the_equations(activation, style, n_layers):
    s = _tiny(activation, n_layers, style)
    w = _weights(s)
    hand = _hand_logits(s, w, TOKENS)
    got = _oracle_logits(s, w, TOKENS)
    for step, (a, b) in enumerate(zip(hand, got)):
        assert b.shape == (s.vocab,)
        assert np.allclose(np.asarray(a), b, rtol=1e-12, atol=1e-13), f"step {step}"
    # greedy pick: the lowest index among the largest logits
    assert int(np.argmax(got[-1])) == max(range(s.vocab), key=lambda i: (hand[-1][i], -i))


def test_without_key_norm_matches_too():
    s = _tiny(qk_norm=False)
    w = _weights(s)
    for a, b in zip(_hand_logits(s, w, TOKENS), _oracle_logits(s, w, TOKENS)):
        assert np.allclose(np.asarray(a), b, rtol=1e-12, atol=1e-13)


def test_first_step_head_output_is_the_value_row():
    # at t = 0 the softmax runs over one key, so h + concat_heads(V_t of the head's group) W_o enters the MLP
    s = _tiny()
    w = _weights(s)
    hand = _hand_logits(s, w, TOKENS[:1], first_step_shortcut=True)[0]
    got = _oracle_logits(s, w, TOKENS[:1], "kvdirect", 0)[0]
    assert np.allclose(np.asarray(hand), got, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("policy,budget", [("kvdirect", 0), ("kvdirect", 1), ("chained", 0), ("chained", 1)])
def test_bounded_policies_match_the_equations(policy, budget):
    s = _tiny(n_layers=2)
    w = _weights(s)
    hand = _hand_logits(s, w, TOKENS + [1, 2])
    got = _oracle_logits(s, w, TOKENS + [1, 2], policy, budget)
    for a, b in zip(hand, got):
        assert np.allclose(np.asarray(a), b, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ the pins have teeth
def _differs(hand, got):
    return max(float(np.max(np.abs(np.asarray(a) - b))) for a, b in zip(hand, got)) > 1e-4


def _mutations():
    def drop_w_o(s, w):
        for lw in w["layers"]:
            lw["w_o"] = [[0.0] * len(r) for r in lw["w_o"]]
        return s, w

    def swap_gate_up(s, w):
        for lw in w["layers"]:
            lw["w_gate"], lw["w_up"] = lw["w_up"], lw["w_gate"]
        return s, w

    def other_activation(s, w):
        return replace(s, activation="silu"), w

    def other_grouping(s, w):
        # interleaved grouping (head a -> KV head a % n_kv) is what the oracle would compute if the
        # query heads were handed over in the order 0, 2, 1, 3: permute W_q's and W_o's head blocks
        dh, perm = s.d_head, [0, 2, 1, 3]
        for lw in w["layers"]:
            lw["w_q"] = [sum((r[p * dh:(p + 1) * dh] for p in perm), []) for r in lw["w_q"]]
        return s, w

    def unit_key_scale(s, w):
        for lw in w["layers"]:
            lw["gamma_k"] = [1.0] * s.d_head
        return s, w

    def unit_mlp_scale(s, w):
        for lw in w["layers"]:
            lw["gamma_mlp"] = [1.0] * s.d_hidden
        return s, w

    def other_pairing(s, w):
        return replace(s, rope_style=ROPE_HALF), w

    def transposed_lm_head(s, w):
        w["lm_head"] = [list(r) for r in zip(*w["lm_head"])]
        return s, w

    def no_final_scale(s, w):
        w["gamma_final"] = [1.0] * s.d_hidden
        return s, w

    return [drop_w_o, swap_gate_up, other_activation, other_grouping, unit_key_scale, unit_mlp_scale,
            other_pairing, transposed_lm_head, no_final_scale]


@pytest.mark.parametrize("mutate", _mutations(), ids=lambda f: f.__name__)
def test_a_wrong_block_is_caught(mutate):
    s = _tiny()
    hand = _hand_logits(s, _weights(s), TOKENS)
    s2, w2 = mutate(s, _weights(s))
    assert _differs(hand, _oracle_logits(s2, w2, TOKENS)), "the hand computation does not see this mistake"
