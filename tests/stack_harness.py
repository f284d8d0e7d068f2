"""Test scaffold: a whole decoder stack driven one token at a time on the GPU (Algorithm 1).

The hot path -- checkpointing residual rows, K/V (re)computation and decode attention -- goes through
the C ABI of the library (include/kvd.h).  Everything around it (embedding lookup, Q projection with
q-norm and rotation, W_o, the gated MLP, the final norm, the vocabulary projection and the greedy
pick) goes through the library's scaffold entry points (include/kvd_scaffold.h): the dense products
run on the same tcgen05 kernel as the K/V projection, the small steps between them are plain kernels.
torch only allocates device memory and copies tensors; no torch arithmetic is on the path.  Both
cache policies share the scaffold line for line.

Cache policies, as in the oracle's stack:
  * "full"      every token's K/V is kept; attention reads one stored segment;
  * "kvdirect"  at most B live K/V entries per layer; the K/V of evicted tokens are rebuilt every
                step from the checkpointed residual rows (kvd_recompute_kv from the store) and
                attention reads [rebuilt, live window incl. current].
  * GpuStackChained: one checkpointed row per token (the row entering layer 0), B live K/V entries
                per layer; every step the evicted prefix is carried through the layers again, layer by
                layer next to the new tokens, so that each layer's K/V of the evicted tokens exist only
                while that layer runs.  This is the variant whose memory is Eq. 24 / Eq. 28.

A row's result in every scaffold step depends on that row alone (the dense products inherit this from
the recompute kernel), so replaying tokens in batches of another size reproduces the first pass bit
for bit -- which the chained variant relies on.
"""
import numpy as np
import torch

import paper_2603_19664_b200 as kvd
from paper_2603_19664_b200.binding import KVD_ACT_GELU_TANH, KVD_ACT_SILU


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
                 layers_stored=None, tiled_attention=False):
        """tiled_attention: every attention call (prefill, decode step, replay) goes through kvd_prefill_attention,
        the tensor-core kernel tiled over query rows, instead of the decode kernels.  Its rows do not depend on the
        batch either, so the bit-identity experiments hold as long as BOTH arms use it."""
        assert policy in ("full", "kvdirect")
        self.tiled = bool(tiled_attention)
        self.s, self.policy, self.budget, self.max_tokens = stack, policy, int(budget), max_tokens
        s = stack
        self.kdim = s.n_kv_heads * s.d_head
        if device_weights:
            self.embed, lm_head, g_final = weights["embed"], weights["lm_head"], weights["gamma_final"]
            self.lw = weights["layers"]
        else:
            self.embed, lm_head, g_final = _dev(weights.embed), _dev(weights.lm_head), _dev(weights.gamma_final)
            self.lw = [{k: _dev(v) for k, v in lw.items()} for lw in weights.layers]
        desc = kvd.make_desc(s.n_layers, s.d_hidden, s.n_q_heads, s.n_kv_heads, s.d_head, s.rms_eps, s.qk_norm,
                             s.rms_eps, s.rope_style, 1, max_tokens, 64)
        self.ctx = ctx = kvd.Kvd(desc)
        self.act = KVD_ACT_SILU if s.activation == "silu" else KVD_ACT_GELU_TANH
        self.lin = []
        for l in range(s.n_layers):
            ls, lw = s.layer_shape(l), self.lw[l]
            ctx.kvd_set_layer(l, lw["w_kv"], lw["gamma_in"], lw.get("gamma_k") if s.qk_norm else None, ls.rope_theta,
                              ls.sliding_window)
            # the scaffold's products, each prepared once: RMSNorm scales folded where a norm precedes the product
            gate_up = torch.cat([lw["w_gate"], lw["w_up"]], dim=1).contiguous()
            self.lin.append({
                "q": ctx.kvd_scaffold_linear_create(lw["w_q"], lw["gamma_in"], s.d_hidden, s.n_q_heads * s.d_head, s.rms_eps),
                "o": ctx.kvd_scaffold_linear_create(lw["w_o"], None, s.n_q_heads * s.d_head, s.d_hidden),
                "gate_up": ctx.kvd_scaffold_linear_create(gate_up, lw["gamma_mlp"], s.d_hidden, 2 * s.d_mlp, s.rms_eps),
                "down": ctx.kvd_scaffold_linear_create(lw["w_down"], None, s.d_mlp, s.d_hidden)})
            del gate_up
        self.lin_head = ctx.kvd_scaffold_linear_create(lm_head, g_final, s.d_hidden, s.vocab, s.rms_eps)
        self.ws = torch.empty(kvd.kvd_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
        ctx.kvd_attach_workspace(self.ws)
        n_stored = s.n_layers if layers_stored is None else layers_stored
        self.arena = torch.empty(kvd.kvd_store_bytes(desc, n_stored), dtype=torch.uint8, device="cuda")
        ctx.kvd_attach_store(self.arena, n_stored)
        # K/V storage indexed by position: the full cache, or the live window of the bounded policy
        self.k_live = [torch.zeros((max_tokens, self.kdim), dtype=torch.bfloat16, device="cuda") for _ in range(s.n_layers)]
        self.v_live = [torch.zeros((max_tokens, self.kdim), dtype=torch.bfloat16, device="cuda") for _ in range(s.n_layers)]
        self.k_old = torch.zeros((max_tokens, self.kdim), dtype=torch.bfloat16, device="cuda")
        self.v_old = torch.zeros((max_tokens, self.kdim), dtype=torch.bfloat16, device="cuda")
        self.win_first = [0] * s.n_layers
        self.t = 0
        self.recomputed_rows = 0
        self.logits_bf16 = None  # [1, padded vocab] of the last token processed

    # ---- scaffold steps (include/kvd_scaffold.h); every tensor made here is an output buffer
    def _linear(self, lin, x):
        m = x.shape[0]
        out = torch.empty((m, lin.out_cols), dtype=torch.bfloat16, device="cuda")
        self.ctx.kvd_scaffold_linear(lin, x, m, out, lin.out_cols)
        return out

    def _embed_rows(self, tokens):
        tok = torch.tensor([int(t) for t in tokens], dtype=torch.int32, device="cuda")
        h = torch.empty((len(tokens), self.s.d_hidden), dtype=torch.bfloat16, device="cuda")
        self.ctx.kvd_scaffold_embed(self.embed, tok, len(tokens), self.s.d_hidden, self.s.vocab, h)
        return h

    def _queries(self, l, h, positions):
        """Normalised, rotated bf16 queries [U, n_q, d_head] of residual rows h [U, d] (Eq. 3)."""
        s, U = self.s, h.shape[0]
        raw = self._linear(self.lin[l]["q"], h)
        pos_t = positions if torch.is_tensor(positions) else torch.tensor(list(positions), dtype=torch.int32, device="cuda")
        q = torch.empty((U, s.n_q_heads, s.d_head), dtype=torch.bfloat16, device="cuda")
        self.ctx.kvd_scaffold_query_finish(l, raw, raw.shape[1], pos_t, U, self.lw[l].get("gamma_q") if s.qk_norm else None, q)
        return q

    def _after_attention(self, l, h, out):
        """W_o, residual add, gated MLP, residual add (Eq. 8-9) for rows h [U, d]; returns the new rows."""
        s, ctx, U = self.s, self.ctx, h.shape[0]
        h = h.clone()
        y = self._linear(self.lin[l]["o"], out.view(U, -1))
        ctx.kvd_scaffold_add_rows(h, y, y.shape[1], U, s.d_hidden)
        gu = self._linear(self.lin[l]["gate_up"], h)
        inner = torch.empty((U, s.d_mlp), dtype=torch.bfloat16, device="cuda")
        ctx.kvd_scaffold_gated_act(gu, gu.shape[1], U, s.d_mlp, self.act, inner)
        y = self._linear(self.lin[l]["down"], inner)
        ctx.kvd_scaffold_add_rows(h, y, y.shape[1], U, s.d_hidden)
        return h

    def _attend(self, l, n, q, positions, positions_dev, segs, out):
        """ATTENTION for n query tokens of the sequence over `segs`: the decode kernels (host loop over launches of at
        most 64 rows) or, with tiled_attention, one launch of the row-tiled tensor-core kernel."""
        if self.tiled:
            self.ctx.kvd_prefill_attention(l, n, q, positions_dev, segs, 0.0, out)
        else:
            self.ctx.kvd_decode_attention_rows(l, n, q, positions, segs, 0.0, out)

    def _logits(self, h_last):
        """Final norm and vocabulary projection of one row; keeps the bf16 logits for greedy_token()."""
        self.logits_bf16 = self._linear(self.lin_head, h_last)
        return self.logits_bf16[0, :self.s.vocab].float()

    def greedy_token(self):
        """Index of the largest logit of the last processed token (lowest index on ties), picked on the GPU."""
        tok = torch.empty((1,), dtype=torch.int32, device="cuda")
        self.ctx.kvd_scaffold_argmax(self.logits_bf16, self.logits_bf16.shape[1], 1, self.s.vocab, tok)
        return int(tok.item())

    def step(self, token):
        s, ctx, pos = self.s, self.ctx, self.t
        assert pos < self.max_tokens
        h = self._embed_rows([token])  # bf16 residual stream
        pos_t = torch.tensor([pos], dtype=torch.int32, device="cuda")
        for l in range(s.n_layers):
            lw, ls = self.lw[l], s.layer_shape(l)
            # scaffold: query
            q = self._queries(l, h, pos_t)
            # hot path, ONE launch: STORE_RESIDUAL of the row entering layer l, K_t, V_t of the current token written at
            # its position in the live storage and, under the bounded policy, RECOMPUTE_KV(C, l) for the evicted tokens
            # this layer still attends to
            kl, vl = self.k_live[l], self.v_live[l]
            lo = 0 if ls.sliding_window == 0 else max(0, pos - ls.sliding_window + 1)
            wf = self.win_first[l] if self.policy == "kvdirect" else 0
            wf = min(wf, pos)
            segs, ranges = [], []
            if self.policy == "kvdirect" and lo < wf:
                n = wf - lo
                ranges = [(0, lo, n, self.k_old, self.v_old)]
                self.recomputed_rows += n
                segs.append((self.k_old, self.v_old, self.kdim, lo, n))
            ctx.kvd_decode_step_kv(l, ranges, self.kdim, h, pos_t, 1, [0], kl[pos:], vl[pos:], self.kdim)
            first_live = max(wf, lo) if self.policy == "kvdirect" else 0
            segs.append((kl[first_live:], vl[first_live:], self.kdim, first_live, pos + 1 - first_live))
            out = torch.empty((1, s.n_q_heads, s.d_head), dtype=torch.bfloat16, device="cuda")
            self._attend(l, 1, q, [pos], pos_t, segs, out)
            # scaffold: W_o, MLP
            h = self._after_attention(l, h, out)
            if self.policy == "kvdirect":
                self.win_first[l] = max(self.win_first[l], pos + 1 - self.budget)  # evict the oldest
        self.t += 1
        return self._logits(h)

    def prefill(self, tokens):
        """Process a whole segment of tokens at once (every token attends to the keys up to its own
        position: the decode-attention call is issued with one "sequence" per segment token).  Returns
        the logits of the last token."""
        s, ctx = self.s, self.ctx
        U, p0 = len(tokens), self.t
        assert p0 + U <= self.max_tokens
        h = self._embed_rows(tokens)  # [U, d] bf16
        positions = list(range(p0, p0 + U))
        pos_t = torch.arange(p0, p0 + U, dtype=torch.int32, device="cuda")
        for l in range(s.n_layers):
            lw, ls = self.lw[l], s.layer_shape(l)
            ctx.kvd_checkpoint_residual(0, l, h, pos_t, U)
            q = self._queries(l, h, pos_t)
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
            self._attend(l, U, q, positions, pos_t, segs, out)
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
            nxt = self.greedy_token()
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

    def __init__(self, stack, weights, budget=0, max_tokens=512, device_weights=False, tiled_attention=False):
        super().__init__(stack, weights, policy="kvdirect", budget=budget, max_tokens=max_tokens,
                         device_weights=device_weights, layers_stored=1, tiled_attention=tiled_attention)
        # the layer-0 rows as the library stores them (documented arena layout)
        self.rows0 = self.arena[:max_tokens * stack.d_hidden * 2].view(torch.bfloat16).view(max_tokens, stack.d_hidden)
        self.replayed_rows = 0

    def step(self, token):
        return self.prefill([int(token)])

    def prefill(self, tokens):
        s, ctx = self.s, self.ctx
        U, p0 = len(tokens), self.t
        assert p0 + U <= self.max_tokens
        h_new = self._embed_rows(tokens)
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
            q_new = self._queries(l, h_new, pos_new_t)
            out_new = torch.empty((U, s.n_q_heads, s.d_head), dtype=torch.bfloat16, device="cuda")
            self._attend(l, U, q_new, pos_new, pos_new_t, segs_new, out_new)
            if N > 0 and l + 1 < s.n_layers:
                # the evicted tokens' own step through this layer: each attends to the evicted keys up
                # to its own position (the position mask does the rest)
                q_old = self._queries(l, h_old, pos_old_t)
                out_old = torch.empty((N, s.n_q_heads, s.d_head), dtype=torch.bfloat16, device="cuda")
                segs_old = [(self.k_old, self.v_old, self.kdim, 0, N)]
                self._attend(l, N, q_old, pos_old, pos_old_t, segs_old, out_old)
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


class BatchStack:
    """A decode batch on a whole stack: `batch` sequences, each with `ctx_len` tokens of context behind it,
    decoding one token per sequence and step under either cache policy from ONE shared state.

    The context is synthetic (the stacks are random-init anyway): every layer's checkpointed residual rows
    are N(0, 1) draws, and the stored K/V of the full-cache arm are those rows' K/V (RECOMPUTE_KV into the
    cache), which is the state Algorithm 1 would have left behind: rows in C, their K/V in the cache.  The
    full-cache arm attends over the stored K/V; the KV-Direct arm keeps the last `window` positions of the
    same buffers as its live window and rebuilds the evicted positions from the rows every step.  Both
    arms share the scaffold, so their tokens must be identical.
    """

    def __init__(self, stack, weights, batch, ctx_len, window, max_steps=8, seed=0):
        self.s, self.batch, self.ctx_len, self.window = stack, batch, ctx_len, window
        s = stack
        self.kdim = s.n_kv_heads * s.d_head
        self.max_tokens = ctx_len + max_steps + 8
        self.embed = weights["embed"]
        self.lw = weights["layers"]
        desc = kvd.make_desc(s.n_layers, s.d_hidden, s.n_q_heads, s.n_kv_heads, s.d_head, s.rms_eps, s.qk_norm,
                             s.rms_eps, s.rope_style, batch, self.max_tokens, batch)
        self.ctx = ctx = kvd.Kvd(desc)
        self.act = KVD_ACT_SILU if s.activation == "silu" else KVD_ACT_GELU_TANH
        self.lin = []
        for l in range(s.n_layers):
            ls, lw = s.layer_shape(l), self.lw[l]
            ctx.kvd_set_layer(l, lw["w_kv"], lw["gamma_in"], lw.get("gamma_k") if s.qk_norm else None, ls.rope_theta,
                              ls.sliding_window)
            gate_up = torch.cat([lw["w_gate"], lw["w_up"]], dim=1).contiguous()
            self.lin.append({
                "q": ctx.kvd_scaffold_linear_create(lw["w_q"], lw["gamma_in"], s.d_hidden, s.n_q_heads * s.d_head, s.rms_eps),
                "o": ctx.kvd_scaffold_linear_create(lw["w_o"], None, s.n_q_heads * s.d_head, s.d_hidden),
                "gate_up": ctx.kvd_scaffold_linear_create(gate_up, lw["gamma_mlp"], s.d_hidden, 2 * s.d_mlp, s.rms_eps),
                "down": ctx.kvd_scaffold_linear_create(lw["w_down"], None, s.d_mlp, s.d_hidden)})
            del gate_up
        self.lin_head = ctx.kvd_scaffold_linear_create(weights["lm_head"], weights["gamma_final"], s.d_hidden, s.vocab,
                                                       s.rms_eps)
        self.ws = torch.empty(kvd.kvd_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
        ctx.kvd_attach_workspace(self.ws)
        self.arena = torch.empty(kvd.kvd_store_bytes(desc, s.n_layers), dtype=torch.uint8, device="cuda")
        ctx.kvd_attach_store(self.arena, s.n_layers)
        mt = self.max_tokens
        self.k_cache = [torch.zeros((batch, mt, self.kdim), dtype=torch.bfloat16, device="cuda") for _ in range(s.n_layers)]
        self.v_cache = [torch.zeros((batch, mt, self.kdim), dtype=torch.bfloat16, device="cuda") for _ in range(s.n_layers)]
        n_old_max = max(ctx_len + max_steps - window, 1)
        self.k_old = torch.zeros((batch, n_old_max, self.kdim), dtype=torch.bfloat16, device="cuda")
        self.v_old = torch.zeros_like(self.k_old)
        # ---- the context: rows into the store, their K/V into the cache
        g = torch.Generator(device="cuda")
        g.manual_seed(3000 + seed)
        pos = torch.arange(ctx_len, dtype=torch.int32, device="cuda")
        self.context_rows = {}  # (layer, seq) -> rows, kept for a few pairs so that tests can check K/V against the oracle
        for l in range(s.n_layers):
            for b in range(batch):
                x = torch.randn((ctx_len, s.d_hidden), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
                ctx.kvd_checkpoint_residual(b, l, x, pos, ctx_len)
                ctx.kvd_recompute_kv(l, None, None, ctx_len, self.k_cache[l][b], self.v_cache[l][b], self.kdim, seq=b,
                                     first_row=0)
                if b in (0, batch - 1) and l in (0, s.n_layers - 1):
                    self.context_rows[(l, b)] = x
        torch.cuda.synchronize()
        # stand-ins for the scaffold's outputs when the hot path is timed by itself (step(..., scaffold=False))
        self.h_fixed = torch.randn((batch, s.d_hidden), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        self.q_fixed = torch.randn((batch, s.n_q_heads, s.d_head), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        self.rows_in_store = ctx_len  # per (layer, sequence); grows with every KV-Direct step
        self.recomputed_rows = 0

    def _linear(self, lin, x):
        m = x.shape[0]
        out = torch.empty((m, lin.out_cols), dtype=torch.bfloat16, device="cuda")
        self.ctx.kvd_scaffold_linear(lin, x, m, out, lin.out_cols)
        return out

    def step(self, tokens_dev, pos, policy, scaffold=True):
        """One decode step of the whole batch at position `pos` (all sequences are equally long).
        tokens_dev: DEVICE int32 [batch].  Returns the next tokens (DEVICE int32 [batch]) picked greedily.
        scaffold=False runs the hot-path launches alone (queries and rows are then whatever the buffers
        hold): used to time the library's part of the step by itself."""
        s, ctx, B, kdim, mt = self.s, self.ctx, self.batch, self.kdim, self.max_tokens
        pos_t = torch.full((B,), pos, dtype=torch.int32, device="cuda")
        qpos = [pos] * B
        h = torch.empty((B, s.d_hidden), dtype=torch.bfloat16, device="cuda")
        if scaffold:
            ctx.kvd_scaffold_embed(self.embed, tokens_dev, B, s.d_hidden, s.vocab, h)
        else:
            h.copy_(self.h_fixed)
        q = torch.empty((B, s.n_q_heads, s.d_head), dtype=torch.bfloat16, device="cuda")
        out = torch.empty_like(q)
        if not scaffold:
            q.copy_(self.q_fixed)
        wf = pos - self.window  # first live position of the KV-Direct arm after the previous step's eviction
        for l in range(s.n_layers):
            ls = s.layer_shape(l)
            kc, vc = self.k_cache[l], self.v_cache[l]
            lo = 0 if ls.sliding_window == 0 else max(0, pos - ls.sliding_window + 1)
            if scaffold:
                raw = self._linear(self.lin[l]["q"], h)
                ctx.kvd_scaffold_query_finish(l, raw, raw.shape[1], pos_t, B, self.lw[l].get("gamma_q") if s.qk_norm else None, q)
            if policy == "kvdirect":
                n_old = max(0, wf - lo)
                ranges = [(b, lo, n_old, self.k_old[b], self.v_old[b]) for b in range(B)] if n_old > 0 else []
                # STORE_RESIDUAL of the new rows, RECOMPUTE_KV for the evicted positions of every sequence and K_t, V_t
                # of the new tokens written straight into the cache rows of the current position: ONE launch
                ctx.kvd_decode_step_kv(l, ranges, kdim, h, pos_t, B, list(range(B)), kc[0, pos], vc[0, pos], mt * kdim)
                self.recomputed_rows += B * n_old
                first_live = max(wf, lo)
                segs = [[(self.k_old[b], self.v_old[b], kdim, lo, n_old),
                         (kc[b, first_live], vc[b, first_live], kdim, first_live, pos + 1 - first_live)] for b in range(B)]
            else:
                ctx.kvd_recompute_kv(l, h, pos_t, B, kc[0, pos], vc[0, pos], mt * kdim)
                segs = [[(kc[b, lo], vc[b, lo], kdim, lo, pos + 1 - lo)] for b in range(B)]
            ctx.kvd_decode_attention(l, B, q, qpos, segs, 0.0, out)
            if scaffold:
                y = self._linear(self.lin[l]["o"], out.view(B, -1))
                ctx.kvd_scaffold_add_rows(h, y, y.shape[1], B, s.d_hidden)
                gu = self._linear(self.lin[l]["gate_up"], h)
                inner = torch.empty((B, s.d_mlp), dtype=torch.bfloat16, device="cuda")
                ctx.kvd_scaffold_gated_act(gu, gu.shape[1], B, s.d_mlp, self.act, inner)
                y = self._linear(self.lin[l]["down"], inner)
                ctx.kvd_scaffold_add_rows(h, y, y.shape[1], B, s.d_hidden)
        nxt = torch.empty((B,), dtype=torch.int32, device="cuda")
        if scaffold:
            self.logits = self._linear(self.lin_head, h)
            ctx.kvd_scaffold_argmax(self.logits, self.logits.shape[1], B, s.vocab, nxt)
        return nxt

    def decode(self, first_tokens, n_steps, policy):
        """n_steps greedy steps from the context state; returns the tokens [n_steps][batch] as lists."""
        assert policy in ("full", "kvdirect")
        if policy == "kvdirect":
            assert self.rows_in_store == self.ctx_len, "the KV-Direct arm appends to the store: run it once, last"
        tok = torch.tensor(first_tokens, dtype=torch.int32, device="cuda")
        outs = []
        for i in range(n_steps):
            tok = self.step(tok, self.ctx_len + i, policy)
            outs.append(tok.tolist())
        if policy == "kvdirect":
            self.rows_in_store += n_steps
        assert self.ctx.kvd_poll_status() == kvd.KVD_OK
        return outs
