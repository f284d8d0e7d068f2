"""The recompute path in fp16 (kvd_set_dtype): the element-type half of the paper's Section 5.1 check.

The reconstruction identities (Eq. 13-14) do not depend on the element type.  With fp16 rows, weights and
outputs:
  * K/V follow the fp64 oracle evaluated on the same fp16-valued inputs (fp16 keeps three more mantissa bits
    than bf16, so the bf16 tolerances hold with room to spare; a tighter relative bound is asserted too);
  * K/V recomputed from checkpointed rows equal, bit for bit, the K/V of the first pass at every length
    16 ... 256 and for single rows (max |dK| = max |dV| = 0), as in bf16;
  * decode attention on fp16 q, K, V follows the oracle too, with bits independent of the segment layout;
  * the fused recompute + attention call on fp16 follows the oracle and the two-call fp16 path;
  * the bf16-only entry points (FP8) refuse an fp16 context.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from kvd_synth import GEMMA3_4B_GLOBAL, QWEN3_4B, SMOLLM2_135M, bf16_to_f64, make_layer_weights, make_residuals

pytestmark = pytest.mark.gpu


def as_f16(bits_bf16: np.ndarray) -> np.ndarray:
    """The synthetic bf16-valued array rounded to fp16 (the values both sides then use)."""
    return bf16_to_f64(bits_bf16).astype(np.float16)


def dev16(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def open_f16(shape, max_tokens, with_store=True):
    w = make_layer_weights(shape)
    desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                         shape.qk_norm, shape.rms_eps, shape.rope_style, 1, max_tokens, 1)
    ctx = kvd.Kvd(desc)
    ctx.kvd_set_dtype(1)
    w16 = {"w_kv": as_f16(w.w_kv), "gamma_in": as_f16(w.gamma_in),
           "gamma_k": as_f16(w.gamma_k) if w.gamma_k is not None else None}
    t = {k: (dev16(v) if v is not None else None) for k, v in w16.items()}
    ctx.kvd_set_layer(0, t["w_kv"], t["gamma_in"], t["gamma_k"], shape.rope_theta, shape.sliding_window)
    if with_store:
        arena = torch.zeros(kvd.kvd_store_bytes(desc, 1), dtype=torch.uint8, device="cuda")
        ctx.kvd_attach_store(arena, 1)
    return ctx, w16


def oracle_f16(shape, w16, X16, pos):
    f = lambda a: None if a is None else a.astype(np.float64)
    return oracle.recompute_kv(f(X16), np.asarray(pos, np.int32), f(w16["gamma_in"]), f(w16["w_kv"]), shape.n_kv_heads,
                               shape.d_head, shape.rms_eps, shape.rope_theta, f(w16["gamma_k"]), shape.rms_eps,
                               shape.rope_style)


@pytest.mark.parametrize("shape,n", [(GEMMA3_4B_GLOBAL, 300), (QWEN3_4B, 130), (SMOLLM2_135M, 200), (GEMMA3_4B_GLOBAL, 1)],
                         ids=lambda v: getattr(v, "name", v))
def test_fp16_recompute_follows_the_oracle(shape, n):
    ctx, w16 = open_f16(shape, 1024)
    kdim = shape.n_kv_heads * shape.d_head
    X16 = as_f16(make_residuals(shape, n, seed=41, outliers=True))
    pos = np.arange(n) + 17
    x, p = dev16(X16), torch.from_numpy(pos.astype(np.int32)).cuda()
    k = torch.full((n + 1, kdim), -7.0, dtype=torch.float16, device="cuda")
    v = torch.full_like(k, -7.0)
    ctx.kvd_recompute_kv(0, x, p, n, k, v, kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.all(k[n:] == -7.0) and torch.all(v[n:] == -7.0)
    Kr, Vr = oracle_f16(shape, w16, X16, pos)
    for name, g, r in (("K", k[:n].cpu().numpy().astype(np.float64), Kr.reshape(n, kdim)),
                       ("V", v[:n].cpu().numpy().astype(np.float64), Vr.reshape(n, kdim))):
        d = g - r
        assert np.max(np.abs(d)) <= 2e-2, name
        # the weights W' = fp16(gamma * W) are rounded once more than the oracle's: relative error stays ~2^-11
        assert np.linalg.norm(d) / np.linalg.norm(r) <= 2e-3, (name, np.linalg.norm(d) / np.linalg.norm(r))


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, SMOLLM2_135M], ids=lambda s: s.name)
def test_fp16_reconstruction_is_bit_exact_at_every_length(shape):
    ctx, w16 = open_f16(shape, 512)
    kdim = shape.n_kv_heads * shape.d_head
    for length in (16, 32, 64, 128, 256):
        X16 = as_f16(make_residuals(shape, length, seed=50 + length, outliers=True))
        pos = np.arange(length)
        x, p = dev16(X16), torch.from_numpy(pos.astype(np.int32)).cuda()
        # first pass: half of the rows in one call, the rest one token at a time (as a decode loop produces them)
        kc = torch.zeros((length, kdim), dtype=torch.float16, device="cuda")
        vc = torch.zeros_like(kc)
        h = length // 2
        ctx.kvd_recompute_kv(0, x[:h], p[:h], h, kc[:h], vc[:h], kdim)
        for m in range(h, length):
            ctx.kvd_recompute_kv(0, x[m:m + 1], p[m:m + 1], 1, kc[m:m + 1], vc[m:m + 1], kdim)
        # checkpoint, then rebuild everything from the store in one launch
        ctx.kvd_reset_sequence(0)
        ctx.kvd_checkpoint_residual(0, 0, x, p, length)
        kr = torch.zeros_like(kc)
        vr = torch.zeros_like(vc)
        ctx.kvd_recompute_kv(0, None, None, length, kr, vr, kdim, seq=0, first_row=0)
        assert ctx.kvd_poll_status() == kvd.KVD_OK
        assert torch.equal(kr.view(torch.int16), kc.view(torch.int16)), length
        assert torch.equal(vr.view(torch.int16), vc.view(torch.int16)), length


def rand_f16(shape_, seed, scale=1.0):
    return (np.random.default_rng(seed).standard_normal(shape_) * scale).astype(np.float16)


@pytest.mark.parametrize("shape,lens", [(GEMMA3_4B_GLOBAL, [1, 300, 2049]), (QWEN3_4B, [700, 5]), (SMOLLM2_135M, [1500])],
                         ids=lambda v: getattr(v, "name", str(v)))
def test_fp16_decode_attention_follows_the_oracle_and_ignores_the_segment_layout(shape, lens):
    """fp16 q, K, V and output on both streaming kernels (fp32 pipes: Gemma shape; mma.sync: Qwen3 and SmolLM2
    shapes): Eq. 6-7 against the fp64 oracle on the same fp16-valued inputs, and identical bits whether the keys
    sit in one segment or in three."""
    import math
    batch = len(lens)
    w = make_layer_weights(shape)
    desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                         shape.qk_norm, shape.rms_eps, shape.rope_style, 1, 4096, batch)
    ctx = kvd.Kvd(desc)
    ctx.kvd_set_dtype(1)
    ctx.kvd_set_layer(0, dev16(as_f16(w.w_kv)), dev16(as_f16(w.gamma_in)),
                      dev16(as_f16(w.gamma_k)) if w.gamma_k is not None else None, shape.rope_theta, shape.sliding_window)
    ws = torch.empty(kvd.kvd_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_workspace(ws)
    kdim = shape.n_kv_heads * shape.d_head
    q16 = rand_f16((batch, shape.n_q_heads, shape.d_head), 1)
    q = dev16(q16)
    Ks = [rand_f16((n, kdim), 10 + b) for b, n in enumerate(lens)]
    Vs = [rand_f16((n, kdim), 20 + b) for b, n in enumerate(lens)]
    kd, vd = [dev16(k) for k in Ks], [dev16(v) for v in Vs]
    q_pos = [n - 1 for n in lens]
    one = [[(kd[b], vd[b], kdim, 0, lens[b])] for b in range(batch)]
    out1 = torch.zeros((batch, shape.n_q_heads, shape.d_head), dtype=torch.float16, device="cuda")
    ctx.kvd_decode_attention(0, batch, q, q_pos, one, 0.0, out1)

    def three(b):
        n = lens[b]
        a, c = n // 3, (2 * n) // 3
        cuts = [(0, a), (a, c), (c, n)]
        return [(kd[b][lo:], vd[b][lo:], kdim, lo, hi - lo) for lo, hi in cuts if hi > lo]
    out3 = torch.zeros_like(out1)
    ctx.kvd_decode_attention(0, batch, q, q_pos, [three(b) for b in range(batch)], 0.0, out3)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.equal(out1.view(torch.int16), out3.view(torch.int16))
    for b, n in enumerate(lens):
        K = Ks[b].astype(np.float64).reshape(n, shape.n_kv_heads, shape.d_head)
        V = Vs[b].astype(np.float64).reshape(n, shape.n_kv_heads, shape.d_head)
        ref = oracle.decode_attention(q16[b].astype(np.float64), q_pos[b], [(K, V, 0)], 1.0 / math.sqrt(shape.d_head),
                                      shape.sliding_window)
        got = out1[b].cpu().numpy().astype(np.float64)
        d = got - ref
        assert np.linalg.norm(d) / np.linalg.norm(ref) <= 1e-2, b
        assert np.max(np.abs(d)) <= 1e-2 * np.max(np.abs(ref)), b


def test_fp16_context_is_refused_by_the_bf16_only_entry_points_and_the_type_is_fixed_once_used():
    shape = GEMMA3_4B_GLOBAL
    ctx, w16 = open_f16(shape, 256)
    with pytest.raises(kvd.KvdError) as e:        # a layer is set: too late to change the type
        ctx.kvd_set_dtype(0)
    assert e.value.status == 5
    x = torch.zeros((2, shape.d_hidden), dtype=torch.float16, device="cuda")
    p = torch.zeros((2,), dtype=torch.int32, device="cuda")
    arena = torch.zeros(kvd.kvd_store_bytes_fp8(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena, 1)
    with pytest.raises(kvd.KvdError) as e:        # the quantiser reads bf16 rows
        ctx.kvd_checkpoint_residual_fp8(0, 0, x, p, 2)
    assert e.value.status == 6
    assert ctx.kvd_poll_status() == kvd.KVD_OK


def test_fp16_kvdirect_layer_equals_the_full_cache_layer_bit_for_bit():
    """Section 5.1 in fp16, one layer: K/V of 300 tokens computed as a decode loop would (first pass), then the
    first 250 evicted and rebuilt from their checkpointed rows; attention over [rebuilt] + [kept] + [current]
    has the bits of attention over the first-pass cache."""
    shape = GEMMA3_4B_GLOBAL
    ctx, w16 = open_f16(shape, 512)
    ws = torch.empty(kvd.kvd_workspace_bytes(ctx.desc), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_workspace(ws)
    kdim = shape.n_kv_heads * shape.d_head
    T, n_old = 300, 250
    X16 = as_f16(make_residuals(shape, T, seed=91, outliers=True))
    x, p = dev16(X16), torch.arange(T, dtype=torch.int32, device="cuda")
    kc = torch.zeros((T, kdim), dtype=torch.float16, device="cuda")
    vc = torch.zeros_like(kc)
    ctx.kvd_recompute_kv(0, x[:200], p[:200], 200, kc, vc, kdim)            # "prefill"
    for m in range(200, T):                                                  # "decode", one token at a time
        ctx.kvd_recompute_kv(0, x[m:m + 1], p[m:m + 1], 1, kc[m:], vc[m:], kdim)
    ctx.kvd_checkpoint_residual(0, 0, x[:n_old], p[:n_old], n_old)
    kr = torch.zeros((n_old, kdim), dtype=torch.float16, device="cuda")
    vr = torch.zeros_like(kr)
    ctx.kvd_recompute_kv(0, None, None, n_old, kr, vr, kdim, seq=0, first_row=0)
    q = dev16(rand_f16((1, shape.n_q_heads, shape.d_head), 5))
    full = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.float16, device="cuda")
    kvdir = torch.zeros_like(full)
    ctx.kvd_decode_attention(0, 1, q, [T - 1], [[(kc, vc, kdim, 0, T)]], 0.0, full)
    ctx.kvd_decode_attention(0, 1, q, [T - 1], [[(kr, vr, kdim, 0, n_old), (kc[n_old:], vc[n_old:], kdim, n_old, T - 1 - n_old),
                                                 (kc[T - 1:], vc[T - 1:], kdim, T - 1, 1)]], 0.0, kvdir)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.equal(kr.view(torch.int16), kc[:n_old].view(torch.int16))
    assert torch.equal(full.view(torch.int16), kvdir.view(torch.int16))
    assert float(full.abs().max()) > 0


def test_element_type_cannot_change_next_to_an_fp8_store():
    # the FP8 entry points quantise bf16 rows and use bf16-folded weights: a context that holds an FP8 store
    # stays bf16 (KVD_ERR_STATE), before any layer is set and whether or not rows are stored yet
    shape = GEMMA3_4B_GLOBAL
    desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps, shape.qk_norm,
                         shape.rms_eps, shape.rope_style, 1, 64, 1)
    ctx = kvd.Kvd(desc)
    ctx.kvd_set_dtype(1)
    ctx.kvd_set_dtype(0)  # nothing holds a type yet: free to change
    arena = torch.zeros(kvd.kvd_store_bytes_fp8(desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena, 1)
    for dt in (1, 2):
        with pytest.raises(kvd.KvdError) as e:
            ctx.kvd_set_dtype(dt)
        assert e.value.status == 5
    ctx.kvd_set_dtype(0)
    ctx.close()


@pytest.mark.parametrize("shape,n_old,n_live", [(GEMMA3_4B_GLOBAL, 600, 40), (QWEN3_4B, 300, 0)], ids=lambda v: getattr(v, "name", v))
def test_fp16_fused_recompute_attention_follows_the_oracle_and_the_two_call_path(shape, n_old, n_live):
    import math
    ctx, w16 = open_f16(shape, 1024)
    ws = torch.empty(kvd.kvd_workspace_bytes(ctx.desc), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_workspace(ws)
    kdim = shape.n_kv_heads * shape.d_head
    T = n_old + n_live + 1
    X16 = as_f16(make_residuals(shape, T, seed=61, outliers=True))
    pos = np.arange(T)
    x, p = dev16(X16), torch.from_numpy(pos.astype(np.int32)).cuda()
    ctx.kvd_checkpoint_residual(0, 0, x[:n_old], p[:n_old], n_old)
    kl = torch.zeros((max(n_live, 1) + 1, kdim), dtype=torch.float16, device="cuda")
    vl = torch.zeros_like(kl)
    if n_live:
        ctx.kvd_recompute_kv(0, x[n_old:n_old + n_live], p[n_old:n_old + n_live], n_live, kl, vl, kdim)
    rng = np.random.Generator(np.random.PCG64(4))
    q16 = rng.standard_normal((1, shape.n_q_heads, shape.d_head)).astype(np.float16)
    q = dev16(q16)
    live = [(kl, vl, kdim, n_old, n_live), (kl[n_live:], vl[n_live:], kdim, T - 1, 1)]
    out_f = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.float16, device="cuda")
    ctx.kvd_decode_attention_recompute(0, 1, q, [T - 1], [(0, 0, n_old)], x[T - 1:], p[T - 1:], 1, kl[n_live:], vl[n_live:],
                                       kdim, [live], 0.0, out_f)
    # the two-call fp16 path on the same inputs
    ko = torch.zeros((n_old, kdim), dtype=torch.float16, device="cuda")
    vo = torch.zeros_like(ko)
    ctx.kvd_recompute_kv(0, None, None, n_old, ko, vo, kdim, seq=0, first_row=0)
    out_t = torch.zeros_like(out_f)
    ctx.kvd_decode_attention(0, 1, q, [T - 1], [[(ko, vo, kdim, 0, n_old)] + live], 0.0, out_t)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    Kr, Vr = oracle_f16(shape, w16, X16, pos)
    ref = oracle.decode_attention(q16[0].astype(np.float64), T - 1, [(Kr, Vr, 0)], 1.0 / math.sqrt(shape.d_head),
                                  shape.sliding_window)
    for name, got in (("fused", out_f), ("two-call", out_t)):
        d = got[0].cpu().numpy().astype(np.float64) - ref
        assert np.linalg.norm(d) / np.linalg.norm(ref) <= 1e-2, name
        assert np.max(np.abs(d)) <= 1e-2 * np.max(np.abs(ref)), name
    ctx.close()
