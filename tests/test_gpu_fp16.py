"""The recompute path in fp16 (kvd_set_dtype): the element-type half of the paper's Section 5.1 check.

The reconstruction identities (Eq. 13-14) do not depend on the element type.  With fp16 rows, weights and
outputs:
  * K/V follow the fp64 oracle evaluated on the same fp16-valued inputs (fp16 keeps three more mantissa bits
    than bf16, so the bf16 tolerances hold with room to spare; a tighter relative bound is asserted too);
  * K/V recomputed from checkpointed rows equal, bit for bit, the K/V of the first pass at every length
    16 ... 256 and for single rows (max |dK| = max |dV| = 0), as in bf16;
  * the entry points that read bf16 K/V refuse an fp16 context.
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


def test_fp16_context_is_refused_where_bf16_is_required_and_the_type_is_fixed_once_used():
    shape = GEMMA3_4B_GLOBAL
    ctx, w16 = open_f16(shape, 256)
    with pytest.raises(kvd.KvdError) as e:        # a layer is set: too late to change the type
        ctx.kvd_set_dtype(0)
    assert e.value.status == 5
    ws = torch.empty(kvd.kvd_workspace_bytes(ctx.desc), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_workspace(ws)
    kdim = shape.n_kv_heads * shape.d_head
    q = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.float16, device="cuda")
    k = torch.zeros((4, kdim), dtype=torch.float16, device="cuda")
    with pytest.raises(kvd.KvdError) as e:
        ctx.kvd_decode_attention(0, 1, q, [3], [[(k, k, kdim, 0, 4)]], 0.0, q)
    assert e.value.status == 6
    assert ctx.kvd_poll_status() == kvd.KVD_OK
