"""Algorithm 1 on a small decoder stack, in fp64 -- TEST INFRASTRUCTURE ONLY.

The model is the paper's pre-norm block (Eq. 3-9): RMSNorm -> Q/K/V projections -> rotation ->
softmax attention -> W_o -> residual add; RMSNorm -> gated MLP -> residual add; then a final
RMSNorm, the vocabulary projection and a greedy argmax (lowest index wins ties).

Three cache policies share every line of the model:
  * ``full``      -- append (K_t, V_t) of every token, never evict;
  * ``kvdirect``  -- keep at most B live entries per layer; the keys and values of evicted tokens
                     are rebuilt each step from the checkpointed residual row that entered the
                     layer (Eq. 13-14), then concatenated [rebuilt, live window, current] as in
                     Algorithm 1.  B = 0 is allowed.
  * ``chained``   -- as ``kvdirect`` but with ONE checkpointed row per token, the row entering
                     layer 0 (the d_hidden * b bytes per token of Eq. 24): every step the evicted
                     tokens are carried through the layers again, so that at layer l their rows
                     h^(l), and from them their keys and values, exist while that layer runs.
K_t and V_t of the token being processed follow the FORWARD equations (Eq. 4-5 with the rotation
of Eq. 11-12), written out here in Python: RMSNorm, one dot product per output channel summed over
the hidden index in ascending order, the per-head key norm, the rotation.  K and V of evicted
tokens come from the RECONSTRUCTION routine (``oracle.recompute_kv``, Eq. 13-14, C).  The two are
separate pieces of code that take the same operations in the same order, which is what
Proposition 3.2 asserts makes them agree bit for bit; the tests check exactly that, so a slip in
either one (a dropped scale, another rotation angle, a transposed weight) shows.

Readings where Algorithm 1 is silent: W_o and the rotations are applied as Eq. 3-8 state; the
current token's (K_t, V_t) joins the live window after attention, then the oldest entries are
evicted while the window exceeds B; the residual row of every token is checkpointed when the token
is first processed, so eviction never needs to look a row up again.  Local (sliding-window) layers
use absolute positions and the mask 0 <= q_pos - key_pos < window.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import math

import numpy as np

from . import ROPE_HALF, ROPE_INTERLEAVED, decode_attention, recompute_kv, rmsnorm, rope  # noqa: F401


def _act(x: np.ndarray, kind: str) -> np.ndarray:
    if kind == "silu":
        return x / (1.0 + np.exp(-x))
    if kind == "gelu_tanh":
        return 0.5 * x * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x + 0.044715 * x ** 3)))
    raise ValueError(kind)


@dataclass
class LayerState:
    rows: List[np.ndarray] = field(default_factory=list)  # checkpointed residual rows, index = position
    win_k: List[np.ndarray] = field(default_factory=list)  # live window keys  [n_kv, d_head] each
    win_v: List[np.ndarray] = field(default_factory=list)
    win_first: int = 0  # position of win_k[0]


class OracleStack:
    """fp64 decoder stack driven one token at a time."""

    def __init__(self, shape, weights_f64: Dict, policy: str = "full", budget: int = 0):
        """``shape`` is a kvd_synth.StackShape-like object; ``weights_f64`` maps
        'embed', 'lm_head', 'gamma_final' and 'layers' (list of dicts) to float64 arrays."""
        assert policy in ("full", "kvdirect", "chained")
        self.s = shape
        self.w = weights_f64
        self.policy = policy
        self.budget = int(budget)
        self.layers = [LayerState() for _ in range(shape.n_layers)]
        self.t = 0  # next position
        self.rows0: List[np.ndarray] = []  # "chained": the one checkpointed row per token
        self.replayed_rows = 0
        self.trace_kv: Optional[List[List]] = None  # when set: per layer list of (K_t, V_t) as first computed

    # -- one token through one layer, given the keys/values before it ------------------------------
    def _block(self, l: int, h: np.ndarray, pos: int, segments_before: List):
        """Eq. 3-9 for the row ``h`` entering layer ``l`` at position ``pos``.  ``segments_before``
        are (K, V, first_pos) runs of the keys at earlier positions.  Returns (row leaving the layer,
        K_t, V_t)."""
        s, lw, ls = self.s, self.w["layers"][l], self.s.layer_shape(l)
        scale = 1.0 / np.sqrt(float(s.d_head))
        xb = rmsnorm(h, lw["gamma_in"], s.rms_eps)
        q = (xb @ lw["w_q"]).reshape(s.n_q_heads, s.d_head)
        for hh in range(s.n_q_heads):
            if s.qk_norm:
                q[hh] = rmsnorm(q[hh], lw["gamma_q"], s.rms_eps)
            q[hh] = rope(q[hh], pos, ls.rope_theta, s.rope_style)
        k_t, v_t = self._kv_forward(l, h, pos)
        heads = decode_attention(q, pos, list(segments_before) + [(k_t, v_t, pos)], scale, ls.sliding_window)
        h = h + heads.reshape(-1) @ lw["w_o"]  # Eq. 8
        xm = rmsnorm(h, lw["gamma_mlp"], s.rms_eps)
        h = h + (_act(xm @ lw["w_gate"], s.activation) * (xm @ lw["w_up"])) @ lw["w_down"]  # Eq. 9
        return h, k_t, v_t

    # -- one decoding step (Algorithm 1) -------------------------------------------------------
    def step(self, token: int) -> np.ndarray:
        s, w = self.s, self.w
        pos = self.t
        h = w["embed"][token].copy()
        chained = self.policy == "chained"
        if chained:
            self.rows0.append(h.copy())  # the only checkpoint: the row entering layer 0
            n_ev = min(self.layers[0].win_first, pos) if self.layers[0].win_k else pos
            ev_rows = [self.rows0[j] for j in range(n_ev)]  # evicted tokens' rows entering the current layer
        for l in range(s.n_layers):
            ls = s.layer_shape(l)
            st = self.layers[l]
            if not chained:
                st.rows.append(h.copy())  # STORE_RESIDUAL: the row entering layer l
            # which past positions does this layer need?
            lo = 0 if ls.sliding_window == 0 else max(0, pos - ls.sliding_window + 1)
            segments = []
            win_lo = st.win_first
            n_win = len(st.win_k)
            if chained:
                if n_ev > 0:
                    k_ev, v_ev = self._kv_rows(l, ev_rows, list(range(n_ev)))  # RECOMPUTE_KV from h^(l)
                    if lo < n_ev:
                        segments.append((k_ev[lo:], v_ev[lo:], lo))
            elif self.policy == "kvdirect":
                old = list(range(lo, min(win_lo, pos))) if n_win > 0 else list(range(lo, pos))
                if old:
                    k_old, v_old = self._kv(l, old)  # RECOMPUTE_KV(C, l)
                    segments.append((k_old, v_old, old[0]))
            if n_win > 0:
                segments.append((np.stack(st.win_k), np.stack(st.win_v), win_lo))
            h, k_t, v_t = self._block(l, h, pos, segments)
            if self.trace_kv is not None:
                self.trace_kv[l].append((k_t[0].copy(), v_t[0].copy()))
            if chained and n_ev > 0 and l + 1 < s.n_layers:
                # the evicted tokens' own step through this layer, in position order: token j sees
                # the evicted keys before it
                ev_rows = [self._block(l, ev_rows[j], j, [(k_ev[:j], v_ev[:j], 0)] if j > 0 else [])[0]
                           for j in range(n_ev)]
                self.replayed_rows += n_ev
            # cache update, then eviction of the oldest entries
            if n_win == 0:
                st.win_first = pos
            st.win_k.append(k_t[0])
            st.win_v.append(v_t[0])
            if self.policy != "full":
                while len(st.win_k) > self.budget:
                    st.win_k.pop(0)
                    st.win_v.pop(0)
                    st.win_first += 1
        self.t += 1
        hf = rmsnorm(h, w["gamma_final"], s.rms_eps)
        return hf @ w["lm_head"]

    def _kv_forward(self, l: int, h: np.ndarray, pos: int):
        """Eq. 4-5 for one token during its own forward pass: K_t = R_pos(keynorm(W_K^T RMSNorm(h))),
        V_t = W_V^T RMSNorm(h), each [1, n_kv, d_head].  Python restatement, independent of the C
        reconstruction routine; every sum runs over its index in ascending order."""
        s, lw, ls = self.s, self.w["layers"][l], self.s.layer_shape(l)
        d, kdim, dh = s.d_hidden, s.n_kv_heads * s.d_head, s.d_head
        ms = 0.0
        for i in range(d):  # Eq. 2
            ms += float(h[i]) * float(h[i])
        r = math.sqrt(ms / d + s.rms_eps)
        xb = [float(h[i]) / r * float(lw["gamma_in"][i]) for i in range(d)]  # Eq. 1
        w_kv = lw["w_kv"]
        acc = np.zeros(2 * kdim, dtype=np.float64)
        for i in range(d):  # Eq. 4-5 before the rotation: channel c receives its terms in ascending i
            acc += xb[i] * w_kv[i]
        k = acc[:kdim].reshape(s.n_kv_heads, dh).copy()
        v = acc[kdim:].reshape(s.n_kv_heads, dh).copy()
        half = dh // 2
        for g in range(s.n_kv_heads):
            if s.qk_norm:
                ss = 0.0
                for j in range(dh):
                    ss += float(k[g, j]) * float(k[g, j])
                rk = math.sqrt(ss / dh + s.rms_eps)
                for j in range(dh):
                    k[g, j] = float(k[g, j]) / rk * float(lw["gamma_k"][j])
            for i in range(half):  # Eq. 11-12, pair i turned by pos * theta^(-2i/d_head)
                phi = float(pos) * math.pow(ls.rope_theta, -2.0 * i / dh)
                c, sn = math.cos(phi), math.sin(phi)
                ia, ib = (i, i + half) if s.rope_style == ROPE_HALF else (2 * i, 2 * i + 1)
                a, b = float(k[g, ia]), float(k[g, ib])
                k[g, ia] = a * c - b * sn
                k[g, ib] = a * sn + b * c
        return k[None], v[None]

    def _kv_rows(self, l: int, rows: List[np.ndarray], positions: List[int]):
        s, lw, ls = self.s, self.w["layers"][l], self.s.layer_shape(l)
        return recompute_kv(np.stack(rows), np.asarray(positions, dtype=np.int32), lw["gamma_in"], lw["w_kv"],
                            s.n_kv_heads, s.d_head, s.rms_eps, ls.rope_theta,
                            lw.get("gamma_k") if s.qk_norm else None, s.rms_eps, s.rope_style)

    def _kv(self, l: int, positions: List[int]):
        st = self.layers[l]
        return self._kv_rows(l, [st.rows[p] for p in positions], positions)

    # -- greedy generation ---------------------------------------------------------------------
    def generate(self, prompt: List[int], n_new: int, forced: Optional[List[int]] = None):
        """Feed the prompt token by token, then decode ``n_new`` tokens greedily.

        Returns (tokens, logits) for the generated part.  ``forced`` (optional) overrides the token
        that is fed back at each generated step (teacher forcing); the argmax is still reported.
        """
        logits = None
        for tok in prompt:
            logits = self.step(int(tok))
        out_tokens, out_logits = [], []
        for i in range(n_new):
            nxt = int(np.argmax(logits))  # numpy returns the lowest index among equal maxima
            out_tokens.append(nxt)
            out_logits.append(logits)
            feed = nxt if forced is None else int(forced[i])
            if i + 1 < n_new:
                logits = self.step(feed)
        return out_tokens, out_logits


def weights_to_f64(sw, widen) -> Dict:
    """Convert a kvd_synth.StackWeights (bf16 bit patterns) to the dict OracleStack expects."""
    return {
        "embed": widen(sw.embed),
        "lm_head": widen(sw.lm_head),
        "gamma_final": widen(sw.gamma_final),
        "layers": [{k: widen(v) for k, v in lw.items()} for lw in sw.layers],
    }
