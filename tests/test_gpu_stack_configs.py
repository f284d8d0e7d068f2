"""The stack-shaped configurations at full size, in the launch shapes bench.py --stack-configs times.

Long context:
Qwen3-4B-shaped layer, batch 8, context 32768, 512 live K/V entries per sequence.

One kvd_recompute_kv_step launch rebuilds 8 x 32256 evicted rows from the residual store together with
the 8 new tokens; one kvd_decode_attention call attends over recomputed + window + current segments.
The oracle checks sampled rows of K/V (first/last rows of tiles, a random sample, several sequences)
and the attention output of two sequences computed from the keys the GPU produced.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from kvd_synth import QWEN3_4B, bf16_to_f64, make_query, make_residuals
from gpu_util import dev, host_f64, kv_errors, open_layer, oracle_kv

pytestmark = pytest.mark.gpu


def test_config4_full_size_sampled():
    shape, batch, ctx_len, budget = QWEN3_4B, 8, 32768, 512
    kdim = shape.n_kv_heads * shape.d_head
    n_old = ctx_len - budget
    ctx, w = open_layer(shape, max_tokens=ctx_len + 8, max_batch=batch, max_seqs=batch, with_store=True)
    X = make_residuals(shape, ctx_len + batch, seed=44)  # the context rows, then one new row per sequence
    x = dev(X)
    pos = torch.arange(ctx_len, dtype=torch.int32, device="cuda")
    for b in range(batch):
        # every sequence checkpoints the same rows shifted by b, so that sequences differ
        ctx.kvd_checkpoint_residual(b, 0, torch.roll(x[:ctx_len], shifts=-b, dims=0).contiguous(), pos, ctx_len)
    Ko = torch.zeros((batch * n_old, kdim), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    kc = torch.zeros((batch, kdim), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    pc = torch.full((batch,), ctx_len, dtype=torch.int32, device="cuda")
    ranges = [(b, 0, n_old, Ko[b * n_old:], Vo[b * n_old:]) for b in range(batch)]
    launches = ctx.kvd_launch_count()
    ctx.kvd_recompute_kv_step(0, ranges, x[ctx_len:], pc, batch, kc, vc, kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert ctx.kvd_launch_count() == launches + 1

    # ---- K/V of sampled rows against the oracle
    rng = np.random.default_rng(4)
    for b in (0, 3, 7):
        rows = np.unique(np.concatenate([[0, 1, 255, 256, 257, n_old - 257, n_old - 256, n_old - 1],
                                         rng.choice(n_old, 40, replace=False)]))
        src = (rows + b) % ctx_len  # the roll above
        Kr, Vr = oracle_kv(shape, w, X[src], rows)
        got_k = host_f64(Ko[b * n_old:(b + 1) * n_old][torch.from_numpy(rows).cuda()])
        got_v = host_f64(Vo[b * n_old:(b + 1) * n_old][torch.from_numpy(rows).cuda()])
        for name, g, r in (("K", got_k, Kr.reshape(len(rows), kdim)), ("V", got_v, Vr.reshape(len(rows), kdim))):
            mx, rel = kv_errors(g, r)
            assert mx <= 2e-2 and rel <= 1e-2, (b, name, mx, rel)
    Kr, Vr = oracle_kv(shape, w, X[ctx_len:], np.full(batch, ctx_len))
    for name, g, r in (("K", host_f64(kc), Kr.reshape(batch, kdim)), ("V", host_f64(vc), Vr.reshape(batch, kdim))):
        mx, rel = kv_errors(g, r)
        assert mx <= 2e-2 and rel <= 1e-2, ("current", name, mx, rel)

    # ---- attention over recomputed + window + current segments (all 8 sequences in one call)
    Kw = torch.randn((batch, budget, kdim), device="cuda").to(torch.bfloat16)
    Vw = torch.randn((batch, budget, kdim), device="cuda").to(torch.bfloat16)
    q_bits = make_query(shape, batch, seed=45)
    q = dev(q_bits)
    out = torch.zeros((batch, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    segs = [[(Ko[b * n_old:], Vo[b * n_old:], kdim, 0, n_old), (Kw[b], Vw[b], kdim, n_old, budget),
             (kc[b:], vc[b:], kdim, ctx_len, 1)] for b in range(batch)]
    ctx.kvd_decode_attention(0, batch, q, [ctx_len] * batch, segs, 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    for b in (0, 7):
        def f64(t):
            return host_f64(t).reshape(-1, shape.n_kv_heads, shape.d_head)
        ref = oracle.decode_attention(bf16_to_f64(q_bits[b]).reshape(shape.n_q_heads, shape.d_head), ctx_len,
                                      [(f64(Ko[b * n_old:(b + 1) * n_old]), f64(Vo[b * n_old:(b + 1) * n_old]), 0),
                                       (f64(Kw[b]), f64(Vw[b]), n_old), (f64(kc[b:b + 1]), f64(vc[b:b + 1]), ctx_len)],
                                      1.0 / math.sqrt(shape.d_head), 0)
        got = host_f64(out[b]).reshape(ref.shape)
        d = got - ref
        assert np.linalg.norm(d) <= 1e-2 * np.linalg.norm(ref)
        assert np.max(np.abs(d)) <= 1e-2 * np.max(np.abs(ref))
    # the same keys from one stored segment per sequence give the same bits
    Kfull = torch.cat([Ko.view(batch, n_old, kdim), Kw, kc.view(batch, 1, kdim)], dim=1).contiguous()
    Vfull = torch.cat([Vo.view(batch, n_old, kdim), Vw, vc.view(batch, 1, kdim)], dim=1).contiguous()
    out1 = torch.zeros_like(out)
    ctx.kvd_decode_attention(0, batch, q, [ctx_len] * batch,
                             [[(Kfull[b], Vfull[b], kdim, 0, ctx_len + 1)] for b in range(batch)], 0.0, out1)
    assert torch.equal(out, out1)
    ctx.close()


@pytest.mark.parametrize("local", [False, True], ids=["global-layer", "local-layer"])
def test_config3_batch64_full_size_sampled(local):
    """The batched decode step of the 34-layer stack configuration at its largest batch: 64 sequences,
    context 2048, 256 live K/V entries; one recompute launch for the 64 evicted ranges and the 64 new
    tokens, one attention call over recomputed + window + current segments."""
    from kvd_synth import GEMMA3_4B_GLOBAL, GEMMA3_4B_LOCAL
    shape = GEMMA3_4B_LOCAL if local else GEMMA3_4B_GLOBAL
    batch, ctx_len, budget = 64, 2048, 256
    kdim = shape.n_kv_heads * shape.d_head
    lo = 0 if shape.sliding_window == 0 else ctx_len - shape.sliding_window + 1
    n_old = ctx_len - budget - lo
    ctx, w = open_layer(shape, max_tokens=ctx_len + 8, max_batch=batch, max_seqs=batch, with_store=True)
    X = make_residuals(shape, ctx_len + batch, seed=46, outliers=True)
    x = dev(X)
    pos = torch.arange(ctx_len, dtype=torch.int32, device="cuda")
    for b in range(batch):
        ctx.kvd_checkpoint_residual(b, 0, torch.roll(x[:ctx_len], shifts=-b, dims=0).contiguous(), pos, ctx_len)
    Ko = torch.zeros((batch * n_old, kdim), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    kc = torch.zeros((batch, kdim), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    pc = torch.full((batch,), ctx_len, dtype=torch.int32, device="cuda")
    ranges = [(b, lo, n_old, Ko[b * n_old:], Vo[b * n_old:]) for b in range(batch)]
    ctx.kvd_recompute_kv_step(0, ranges, x[ctx_len:], pc, batch, kc, vc, kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    rng = np.random.default_rng(5)
    for b in (0, 31, 63):
        rows = np.unique(np.concatenate([[0, 1, 255, 256, n_old - 1], rng.choice(n_old, 30, replace=False)]))
        src = (rows + lo + b) % ctx_len
        Kr, Vr = oracle_kv(shape, w, X[src], rows + lo)
        idx = torch.from_numpy(rows).cuda()
        for name, g, r in (("K", host_f64(Ko[b * n_old:(b + 1) * n_old][idx]), Kr.reshape(len(rows), kdim)),
                           ("V", host_f64(Vo[b * n_old:(b + 1) * n_old][idx]), Vr.reshape(len(rows), kdim))):
            mx, rel = kv_errors(g, r)
            assert mx <= 2e-2 and rel <= 1e-2, (b, name, mx, rel)
    wf = ctx_len - budget
    Kw = torch.randn((batch, budget, kdim), device="cuda").to(torch.bfloat16)
    Vw = torch.randn((batch, budget, kdim), device="cuda").to(torch.bfloat16)
    q_bits = make_query(shape, batch, seed=47)
    q = dev(q_bits)
    out = torch.zeros((batch, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    segs = [[(Ko[b * n_old:], Vo[b * n_old:], kdim, lo, n_old), (Kw[b], Vw[b], kdim, wf, budget),
             (kc[b:], vc[b:], kdim, ctx_len, 1)] for b in range(batch)]
    ctx.kvd_decode_attention(0, batch, q, [ctx_len] * batch, segs, 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK

    def f64(t):
        return host_f64(t).reshape(-1, shape.n_kv_heads, shape.d_head)
    for b in (0, 17, 63):
        ref = oracle.decode_attention(bf16_to_f64(q_bits[b]).reshape(shape.n_q_heads, shape.d_head), ctx_len,
                                      [(f64(Ko[b * n_old:(b + 1) * n_old]), f64(Vo[b * n_old:(b + 1) * n_old]), lo),
                                       (f64(Kw[b]), f64(Vw[b]), wf), (f64(kc[b:b + 1]), f64(vc[b:b + 1]), ctx_len)],
                                      1.0 / math.sqrt(shape.d_head), shape.sliding_window)
        d = host_f64(out[b]).reshape(ref.shape) - ref
        assert np.linalg.norm(d) <= 1e-2 * np.linalg.norm(ref)
        assert np.max(np.abs(d)) <= 1e-2 * np.max(np.abs(ref))
    ctx.close()


def test_config3_layers_at_full_shape_tokens_match_across_policies():
    """Six layers (one local/global period) of the Gemma-3-4B-shaped stack at full width -- hidden 2560, MLP
    10240, vocabulary 262144 -- decoding a batch from a 2048-token context with a 256-token window: the
    KV-Direct arm (evicted K/V rebuilt every step) must pick the same tokens as the full-cache arm, the cached
    context K/V must follow the oracle on sampled rows, and nothing but the library's kernels computes."""
    import sys, os
    from dataclasses import replace
    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    from kvd_synth import GEMMA3_4B_STACK, LayerWeights
    from stack_harness import BatchStack, torch_stack_weights
    stack = replace(GEMMA3_4B_STACK, n_layers=6, name="gemma3-4b-6l")
    w = torch_stack_weights(stack, seed=3)
    batch, ctx_len, window, steps = 3, 2048, 256, 4
    m = BatchStack(stack, w, batch, ctx_len, window, max_steps=steps)
    first = [11, 222222, 3333]
    launches = m.ctx.kvd_launch_count()
    full = m.decode(first, steps, "full")
    per_step_full = (m.ctx.kvd_launch_count() - launches) // steps
    kvdir = m.decode(first, steps, "kvdirect")
    assert full == kvdir
    assert len({t for row in full for t in row}) > 3, "degenerate generation would prove nothing"
    # evicted rows rebuilt per step: 5 local layers see 1024 - 257 of them, the global layer 2048 - 256
    assert m.recomputed_rows >= batch * steps * (5 * (1024 - 257) + (2048 - 256))
    assert per_step_full >= 6 * 9  # every layer: query product + finish, K_t/V_t, attention (2), W_o, add, gate/up, act, down, add
    # ---- cached context K/V against the oracle, sampled rows of the first and last layer
    rng = np.random.default_rng(5)
    kdim = stack.n_kv_heads * stack.d_head
    for (l, b), x in m.context_rows.items():
        ls = stack.layer_shape(l)
        rows = np.unique(np.concatenate([[0, 1, 255, 256, ctx_len - 1], rng.choice(ctx_len, 12, replace=False)]))
        lw = w["layers"][l]
        wts = LayerWeights(*(t.cpu().view(torch.int16).numpy().view(np.uint16) for t in (lw["w_kv"], lw["gamma_in"], lw["gamma_k"])))
        X = x[torch.from_numpy(rows).cuda()].cpu().view(torch.int16).numpy().view(np.uint16)
        Kr, Vr = oracle_kv(ls, wts, X, rows)
        got_k = host_f64(m.k_cache[l][b][torch.from_numpy(rows).cuda()])
        got_v = host_f64(m.v_cache[l][b][torch.from_numpy(rows).cuda()])
        for name, g, r in (("K", got_k, Kr.reshape(len(rows), kdim)), ("V", got_v, Vr.reshape(len(rows), kdim))):
            mx, rel = kv_errors(g, r)
            assert mx <= 2e-2 and rel <= 1e-2, (l, b, name, mx, rel)
    m.ctx.close()
