"""Test scaffold: a whole decoder stack driven one token at a time on the GPU (Algorithm 1).

The hot path -- checkpointing residual rows, K/V (re)computation and decode attention -- goes through
the C ABI of the library.  Everything around it (embedding lookup, Q projection with q-norm and
rotation, W_o, the gated MLP, the final norm, the vocabulary projection and the argmax) is plain
torch arithmetic: it is scaffolding that both cache policies share line for line, needed only to
produce realistic residual streams and to turn attention outputs into tokens.

Cache policies, as in the oracle's stack:
  * "full"      every token's K/V is kept; attention reads one stored segment;
  * "kvdirect"  at most B live K/V entries per layer; the K/V of evicted tokens are rebuilt every
                step from the checkpointed residual rows (kvd_recompute_kv from the store) and
                attention reads [rebuilt, live window incl. current].
  * GpuStackChained: one checkpointed row per token (the row entering layer 0), B live K/V entries
                per layer; every step the evicted prefix is carried through the layers again, layer by
                layer next to the new tokens, so that each layer's K/V of the evicted tokens exist only
                while that layer runs.  This is the variant whose memory is Eq. 24 / Eq. 28.

`exact_scaffold=True` makes the scaffold's matrix products and norms accumulate in fp64 before
rounding to bf16: their bf16 results then do not depend on how many rows are processed at once
(the library's kernels have that property by construction), which the chained variant needs to
reproduce the first pass bit for bit when it replays tokens in different batches.
"""
import math

import numpy as np
import torch

import paper_2603_19664_b200 as kvd
from kvd_synth import ROPE_HALF


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def torch_stack_weights(stack, seed=0):
    """Random-init weights of a (possibly full-size) stack drawn on the GPU with torch: N(0, 0.02)
    matrices, N(0, 1) embeddings, norm scales 1 + N(0, 0.02).  Returns device tensors in the layout
    GpuStack expects (use with `device_weights=True`)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(1000 + seed)

    def rn(shape, std, mean=0.0):
        return (torch.randn(shape, generator=g, device="cuda", dtype=torch.float32) * std + mean).to(torch.bfloat16)

    s = stack
    nq, nkv, dh, d = s.n_q_heads, s.n_kv_heads, s.d_head, s.d_hidden
    layers = []
    for _ in range(s.n_layers):
        lw = {"w_kv": rn((d, 2 * nkv * dh), 0.02), "w_q": rn((d, nq * dh), 0.02), "w_o": rn((nq * dh, d), 0.02),
              "w_gate": rn((d, s.d_mlp), 0.02), "w_up": rn((d, s.d_mlp), 0.02), "w_down": rn((s.d_mlp, d), 0.02),
              "gamma_in": rn((d,), 0.02, 1.0), "gamma_mlp": rn((d,), 0.02, 1.0)}
        if s.qk_norm:
            lw["gamma_q"] = rn((dh,), 0.02, 1.0)
            lw["gamma_k"] = rn((dh,), 0.02, 1.0)
        layers.append(lw)
    return {"embed": rn((s.vocab, d), 1.0), "lm_head": rn((d, s.vocab), 0.02), "gamma_final": rn((d,), 0.02, 1.0),
            "layers": layers}


class GpuStack:
    def __init__(self, stack, weights, policy="full", budget=0, max_tokens=512, device_weights=False,
                 exact_scaffold=False, layers_stored=None):
        assert policy in ("full", "kvdirect")
        self.s, self.policy, self.budget, self.max_tokens = stack, policy, int(budget), max_tokens
        self.exact = bool(exact_scaffold)
        s = stack
        self.kdim = s.n_kv_heads * s.d_head
        if device_weights:
            self.embed, self.lm_head = weights["embed"], weights["lm_head"]
            self.g_final = weights["gamma_final"].float()
            self.lw = weights["layers"]
        else:
            self.embed = _dev(weights.embed)
            self.lm_head = _dev(weights.lm_head)
            self.g_final = _dev(weights.gamma_final).float()
            self.lw = []
            for lw in weights.layers:
                d = {k: _dev(v) for k, v in lw.items()}
                self.lw.append(d)
        desc = kvd.make_desc(s.n_layers, s.d_hidden, s.n_q_heads, s.n_kv_heads, s.d_head, s.rms_eps, s.qk_norm,
                             s.rms_eps, s.rope_style, 1, max_tokens, 64)
        self.ctx = kvd.Kvd(desc)
        for l in range(s.n_layers):
            ls = s.layer_shape(l)
            self.ctx.kvd_set_layer(l, self.lw[l]["w_kv"], self.lw[l]["gamma_in"],
                                   self.lw[l].get("gamma_k") if s.qk_norm else None, ls.rope_theta, ls.sliding_window)
        self.ws = torch.empty(kvd.kvd_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
        self.ctx.kvd_attach_workspace(self.ws)
        n_stored = s.n_layers if layers_stored is None else layers_stored
        self.arena = torch.empty(kvd.kvd_store_bytes(desc, n_stored), dtype=torch.uint8, device="cuda")
        self.ctx.kvd_attach_store(self.arena, n_stored)
        # K/V storage indexed by position: the full cache, or the live window of the bounded policy
        self.k_live = [torch.zeros((max_tokens, self.kdim), dtype=torch.bfloat16, device="cuda") for _ in range(s.n_layers)]
        self.v_live = [torch.zeros((max_tokens, self.kdim), dtype=torch.bfloat16, device="cuda") for _ in range(s.n_layers)]
        self.k_old = torch.zeros((max_tokens, self.kdim), dtype=torch.bfloat16, device="cuda")
        self.v_old = torch.zeros((max_tokens, self.kdim), dtype=torch.bfloat16, device="cuda")
        self.win_first = [0] * s.n_layers
        self.t = 0
        self.recomputed_rows = 0
        # rotation angles for q (scaffold side), fp64 on the host like the library's tables
        self.inv_freq = {}

    def _rms(self, x, gamma):
        if self.exact:
            xd = x.double()
            return (xd * torch.rsqrt(xd.pow(2).mean(-1, keepdim=True) + self.s.rms_eps) * gamma.double()).float()
        xf = x.float()
        return xf * torch.rsqrt(xf.pow(2).mean(-1, keepdim=True) + self.s.rms_eps) * gamma.float()

    def _mm(self, x, w):
        """bf16 x @ bf16 w -> bf16 (fp64 accumulation when exact_scaffold)."""
        if self.exact:
            return (x.double() @ w.double()).to(torch.bfloat16)
        return x @ w

    def _qnorm(self, q, gamma_q):
        if self.exact:
            qd = q.double()
            return (qd * torch.rsqrt(qd.pow(2).mean(-1, keepdim=True) + self.s.rms_eps) * gamma_q.double()).float()
        return q * torch.rsqrt(q.pow(2).mean(-1, keepdim=True) + self.s.rms_eps) * gamma_q.float()

    def _queries(self, l, h, positions):
        """Scaffold: normalised, rotated bf16 queries [U, n_q, d_head] of residual rows h [U, d]."""
        s, lw, ls = self.s, self.lw[l], self.s.layer_shape(l)
        xb = self._rms(h, lw["gamma_in"]).to(torch.bfloat16)
        q = self._mm(xb, lw["w_q"]).float().view(h.shape[0], s.n_q_heads, s.d_head)
        if s.qk_norm:
            q = self._qnorm(q, lw["gamma_q"])
        return self._rope_q(q, positions, ls.rope_theta).to(torch.bfloat16).contiguous()

    def _after_attention(self, l, h, out):
        """Scaffold: W_o, residual add, gated MLP, residual add (Eq. 8-9) for rows h [U, d]."""
        lw = self.lw[l]
        h = (h.float() + self._mm(out.view(h.shape[0], -1), lw["w_o"]).float()).to(torch.bfloat16)
        xm = self._rms(h, lw["gamma_mlp"]).to(torch.bfloat16)
        gate = self._act(self._mm(xm, lw["w_gate"]).float()) * self._mm(xm, lw["w_up"]).float()
        mlp = self._mm(gate.to(torch.bfloat16), lw["w_down"])
        return (h.float() + mlp.float()).to(torch.bfloat16)

    def _rope_q(self, q, pos, theta):
        """q: [..., n_q, d_head] with `pos` an int or a list of positions (one per leading row)."""
        s = self.s
        half = s.d_head // 2
        key = float(theta)
        if key not in self.inv_freq:
            self.inv_freq[key] = torch.tensor([theta ** (-2.0 * i / s.d_head) for i in range(half)], dtype=torch.float64)
        if isinstance(pos, int):
            ang = (self.inv_freq[key] * pos)
        else:
            ang = torch.tensor(pos, dtype=torch.float64)[:, None, None] * self.inv_freq[key]  # [U, 1, half]
        c, sn = torch.cos(ang).float().cuda(), torch.sin(ang).float().cuda()
        if s.rope_style == ROPE_HALF:
            a, b = q[..., :half], q[..., half:]
            return torch.cat([a * c - b * sn, a * sn + b * c], dim=-1)
        a, b = q[..., 0::2], q[..., 1::2]
        out = torch.empty_like(q)
        out[..., 0::2] = a * c - b * sn
        out[..., 1::2] = a * sn + b * c
        return out

    def _act(self, x):
        if self.s.activation == "silu":
            return torch.nn.functional.silu(x)
        return torch.nn.functional.gelu(x, approximate="tanh")

    def step(self, token):
        s, ctx, pos = self.s, self.ctx, self.t
        assert pos < self.max_tokens
        h = self.embed[token].clone().view(1, -1)  # bf16 residual stream
        pos_t = torch.tensor([pos], dtype=torch.int32, device="cuda")
        for l in range(s.n_layers):
            lw, ls = self.lw[l], s.layer_shape(l)
            ctx.kvd_checkpoint_residual(0, l, h, pos_t, 1)  # STORE_RESIDUAL: the row entering layer l
            # scaffold: query
            q = self._queries(l, h, [pos])
            # hot path: K_t, V_t of the current token, written at its position in the live storage
            kl, vl = self.k_live[l], self.v_live[l]
            lo = 0 if ls.sliding_window == 0 else max(0, pos - ls.sliding_window + 1)
            wf = self.win_first[l] if self.policy == "kvdirect" else 0
            wf = min(wf, pos)
            segs = []
            if self.policy == "kvdirect" and lo < wf:
                # evicted tokens this layer still attends to: RECOMPUTE_KV(C, l), in the same launch
                # as K_t, V_t of the current token
                n = wf - lo
                ctx.kvd_recompute_kv_step(l, [(0, lo, n, self.k_old, self.v_old)], h, pos_t, 1, kl[pos:], vl[pos:],
                                          self.kdim)
                self.recomputed_rows += n
                segs.append((self.k_old, self.v_old, self.kdim, lo, n))
            else:
                ctx.kvd_recompute_kv(l, h, pos_t, 1, kl[pos:], vl[pos:], self.kdim)
            first_live = max(wf, lo) if self.policy == "kvdirect" else 0
            segs.append((kl[first_live:], vl[first_live:], self.kdim, first_live, pos + 1 - first_live))
            out = torch.empty((1, s.n_q_heads, s.d_head), dtype=torch.bfloat16, device="cuda")
            ctx.kvd_decode_attention(l, 1, q, [pos], [segs], 0.0, out)
            # scaffold: W_o, MLP
            h = self._after_attention(l, h, out)
            if self.policy == "kvdirect":
                self.win_first[l] = max(self.win_first[l], pos + 1 - self.budget)  # evict the oldest
        self.t += 1
        return self._logits(h)

    def _logits(self, h_last):
        hf = self._rms(h_last, self.g_final).to(torch.bfloat16)
        return self._mm(hf, self.lm_head).float().view(-1)

    def prefill(self, tokens):
        """Process a whole segment of tokens at once (every token attends to the keys up to its own
        position: the decode-attention call is issued with one "sequence" per segment token).  Returns
        the logits of the last token."""
        s, ctx = self.s, self.ctx
        U, p0 = len(tokens), self.t
        assert p0 + U <= self.max_tokens
        tok = torch.tensor(tokens, dtype=torch.long, device="cuda")
        h = self.embed[tok].clone()  # [U, d] bf16
        positions = list(range(p0, p0 + U))
        pos_t = torch.arange(p0, p0 + U, dtype=torch.int32, device="cuda")
        for l in range(s.n_layers):
            lw, ls = self.lw[l], s.layer_shape(l)
            ctx.kvd_checkpoint_residual(0, l, h, pos_t, U)
            q = self._queries(l, h, positions)
            kl, vl = self.k_live[l], self.v_live[l]
            ctx.kvd_recompute_kv(l, h, pos_t, U, kl[p0:], vl[p0:], self.kdim)
            lo_min = 0 if ls.sliding_window == 0 else max(0, p0 - ls.sliding_window + 1)
            wf = min(self.win_first[l], p0) if self.policy == "kvdirect" else 0
            segs = []
            if self.policy == "kvdirect" and lo_min < wf:
                n = wf - lo_min
                ctx.kvd_recompute_kv(l, None, None, n, self.k_old, self.v_old, self.kdim, seq=0, first_row=lo_min)
                self.recomputed_rows += n
                segs.append((self.k_old, self.v_old, self.kdim, lo_min, n))
            first_live = max(wf, lo_min) if self.policy == "kvdirect" else 0
            segs.append((kl[first_live:], vl[first_live:], self.kdim, first_live, p0 + U - first_live))
            out = torch.empty((U, s.n_q_heads, s.d_head), dtype=torch.bfloat16, device="cuda")
            for b0 in range(0, U, 64):
                nb = min(64, U - b0)
                ctx.kvd_decode_attention(l, nb, q[b0:], positions[b0:b0 + nb], [segs] * nb, 0.0, out[b0:])
            h = self._after_attention(l, h, out)
            if self.policy == "kvdirect":
                self.win_first[l] = max(self.win_first[l], p0 + U - self.budget)
        self.t += U
        return self._logits(h[-1:])

    def generate(self, prompt, n_new, forced=None):
        logits = None
        for tok in prompt:
            logits = self.step(int(tok))
        toks, lgs = [], []
        for i in range(n_new):
            nxt = int(torch.argmax(logits).item())
            toks.append(nxt)
            lgs.append(logits.clone())
            if i + 1 < n_new:
                logits = self.step(nxt if forced is None else int(forced[i]))
        assert self.ctx.kvd_poll_status() == kvd.KVD_OK
        return toks, lgs

    def memory_report(self):
        """Bytes the policy needs (Eq. 28 accounting next to what per-layer checkpoints cost)."""
        s, T, B = self.s, self.t, self.budget
        kv_tok = 2 * s.n_kv_heads * s.d_head * 2
        live = T if self.policy == "full" else min(B, T)
        return {"tokens": T, "live_kv_bytes": s.n_layers * live * kv_tok,
                "checkpoint_bytes_per_layer_rows": self.ctx.kvd_memory_stats()["checkpoint_bytes_used"],
                "eq28_bytes": 2 * min(B, T) * s.n_layers * s.n_kv_heads * s.d_head * 2 + max(T - B, 0) * s.d_hidden * 2,
                "full_cache_bytes": s.n_layers * T * kv_tok}


class GpuStackChained(GpuStack):
    """One checkpointed residual row per token (the row entering layer 0) and a window of B live K/V
    entries per layer.  Every call carries the evicted prefix [0, first live position) through the
    layers again next to the new tokens: at layer l the K/V of the evicted tokens are recomputed from
    their current rows (the same kvd_recompute_kv as ever), serve the new tokens' attention and the
    evicted tokens' own causal attention, and are dropped when the rows move on to layer l + 1."""

    def __init__(self, stack, weights, budget=0, max_tokens=512, device_weights=False, exact_scaffold=True):
        super().__init__(stack, weights, policy="kvdirect", budget=budget, max_tokens=max_tokens,
                         device_weights=device_weights, exact_scaffold=exact_scaffold, layers_stored=1)
        # the layer-0 rows as the library stores them (documented arena layout)
        self.rows0 = self.arena[:max_tokens * stack.d_hidden * 2].view(torch.bfloat16).view(max_tokens, stack.d_hidden)
        self.replayed_rows = 0

    def step(self, token):
        return self.prefill([int(token)])

    def prefill(self, tokens):
        s, ctx = self.s, self.ctx
        U, p0 = len(tokens), self.t
        assert p0 + U <= self.max_tokens
        tok = torch.tensor(tokens, dtype=torch.long, device="cuda")
        h_new = self.embed[tok].clone()
        pos_new = list(range(p0, p0 + U))
        pos_new_t = torch.arange(p0, p0 + U, dtype=torch.int32, device="cuda")
        ctx.kvd_checkpoint_residual(0, 0, h_new, pos_new_t, U)  # STORE_RESIDUAL: one row per token
        N = min(self.win_first[0], p0)  # evicted prefix [0, N); the windows of all layers move together
        h_old = self.rows0[:N].clone() if N > 0 else None
        pos_old = list(range(N))
        pos_old_t = torch.arange(N, dtype=torch.int32, device="cuda")
        for l in range(s.n_layers):
            ls = s.layer_shape(l)
            kl, vl = self.k_live[l], self.v_live[l]
            ctx.kvd_recompute_kv(l, h_new, pos_new_t, U, kl[p0:], vl[p0:], self.kdim)
            segs_new = []
            if N > 0:
                # RECOMPUTE_KV for the evicted tokens from their rows as they enter this layer
                ctx.kvd_recompute_kv(l, h_old, pos_old_t, N, self.k_old, self.v_old, self.kdim)
                self.recomputed_rows += N
                segs_new.append((self.k_old, self.v_old, self.kdim, 0, N))
            segs_new.append((kl[N:], vl[N:], self.kdim, N, p0 + U - N))
            q_new = self._queries(l, h_new, pos_new)
            out_new = torch.empty((U, s.n_q_heads, s.d_head), dtype=torch.bfloat16, device="cuda")
            for b0 in range(0, U, 64):
                nb = min(64, U - b0)
                ctx.kvd_decode_attention(l, nb, q_new[b0:], pos_new[b0:b0 + nb], [segs_new] * nb, 0.0, out_new[b0:])
            if N > 0 and l + 1 < s.n_layers:
                # the evicted tokens' own step through this layer: each attends to the evicted keys up
                # to its own position (the position mask does the rest)
                q_old = self._queries(l, h_old, pos_old)
                out_old = torch.empty((N, s.n_q_heads, s.d_head), dtype=torch.bfloat16, device="cuda")
                segs_old = [(self.k_old, self.v_old, self.kdim, 0, N)]
                for b0 in range(0, N, 64):
                    nb = min(64, N - b0)
                    ctx.kvd_decode_attention(l, nb, q_old[b0:], pos_old[b0:b0 + nb], [segs_old] * nb, 0.0, out_old[b0:])
                h_old = self._after_attention(l, h_old, out_old)
                self.replayed_rows += N
            h_new = self._after_attention(l, h_new, out_new)
        for l in range(s.n_layers):
            self.win_first[l] = max(self.win_first[l], p0 + U - self.budget)
        self.t += U
        return self._logits(h_new[-1:])

    def memory_report(self):
        rep = super().memory_report()
        rep["checkpoint_bytes_single_row"] = rep.pop("checkpoint_bytes_per_layer_rows")
        return rep
