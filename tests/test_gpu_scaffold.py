"""The scaffold entry points (include/kvd_scaffold.h) against plain fp64 definitions.

These calls are not part of the method; they exist so that whole-stack runs (Algorithm 1 around the hot
path: Eq. 3, 8, 9, final norm, vocabulary projection, greedy pick) use the library's own kernels.  Each is
compared here with its definition written out in numpy / the oracle's RMSNorm and rotation, and the dense
product is checked for the property the chained-recompute stack relies on: a row's output bits do not
depend on how many rows the call carries.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from paper_2603_19664_b200.binding import KVD_ACT_GELU_TANH, KVD_ACT_SILU
from kvd_synth import GEMMA3_4B_GLOBAL, QWEN3_4B, SMOLLM2_135M, bf16_to_f64, f32_to_bf16_bits
from gpu_util import dev, host_bits, host_f64, open_layer

pytestmark = pytest.mark.gpu


def _bits(rng, shape, std, mean=0.0):
    return f32_to_bf16_bits(rng.standard_normal(size=shape, dtype=np.float32) * np.float32(std) + np.float32(mean))


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, SMOLLM2_135M], ids=lambda s: s.name)
@pytest.mark.parametrize("k,n,m,norm", [(256, 512, 5, True), (192, 200, 300, True), (640, 1280, 70, False),
                                         (2560, 2048, 33, True), (1024, 96, 1, False)])
def test_linear_matches_its_definition(shape, k, n, m, norm):
    ctx, _ = open_layer(shape, max_tokens=512)
    rng = np.random.Generator(np.random.PCG64(11 + k + n))
    W, X, G = _bits(rng, (k, n), 0.05), _bits(rng, (m, k), 1.0), _bits(rng, (k,), 0.1, 1.0)
    eps = 1e-5
    lin = ctx.kvd_scaffold_linear_create(dev(W), dev(G) if norm else None, k, n, eps)
    assert lin.out_cols >= n and lin.out_cols % 128 == 0
    out = torch.full((m, lin.out_cols + 8), 7.0, dtype=torch.bfloat16, device="cuda")
    ctx.kvd_scaffold_linear(lin, dev(X), m, out, lin.out_cols + 8)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    x, w = bf16_to_f64(X), bf16_to_f64(W)
    if norm:
        # the product reads W' = bf16(gamma * W) and scales the rows by 1/rms afterwards
        wp = bf16_to_f64(f32_to_bf16_bits((bf16_to_f64(G)[:, None] * w).astype(np.float32)))
        ref = (x @ wp) / np.sqrt(np.mean(x * x, axis=1, keepdims=True) + eps)
        # ... which is RMSNorm (Eq. 1-2) ahead of the product, up to the rounding of W'
        ref2 = np.stack([oracle.rmsnorm(x[r], bf16_to_f64(G), eps) for r in range(m)]) @ w
        assert np.linalg.norm(ref - ref2) <= 4e-3 * np.linalg.norm(ref2)
    else:
        ref = x @ w
    got = host_f64(out)
    assert np.linalg.norm(got[:, :n] - ref) <= 4e-3 * np.linalg.norm(ref)  # bf16 output rounding: 2^-9 per element
    assert np.max(np.abs(got[:, :n] - ref)) <= 2 ** -8 * np.max(np.abs(ref)) + 1e-6
    assert np.all(got[:, n:lin.out_cols] == 0.0)          # padding columns of the tile
    assert np.all(got[:, lin.out_cols:] == 7.0)           # beyond the tile: untouched
    ctx.close()


def test_linear_row_bits_do_not_depend_on_the_batch():
    shape = QWEN3_4B
    ctx, _ = open_layer(shape, max_tokens=1024)
    rng = np.random.Generator(np.random.PCG64(5))
    k, n = 2560, 768
    W, X, G = _bits(rng, (k, n), 0.02), _bits(rng, (600, k), 1.0), _bits(rng, (k,), 0.02, 1.0)
    lin = ctx.kvd_scaffold_linear_create(dev(W), dev(G), k, n, 1e-6)
    x = dev(X)
    big = torch.empty((600, lin.out_cols), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_scaffold_linear(lin, x, 600, big, lin.out_cols)          # statistics by the kernel of their own
    for r0, m in ((0, 1), (17, 3), (255, 64), (300, 65), (599, 1)):  # ... and inside the main kernel (<= 64 rows)
        small = torch.empty((m, lin.out_cols), dtype=torch.bfloat16, device="cuda")
        ctx.kvd_scaffold_linear(lin, x[r0:r0 + m], m, small, lin.out_cols)
        assert torch.equal(small, big[r0:r0 + m]), (r0, m)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    ctx.close()


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, QWEN3_4B, SMOLLM2_135M], ids=lambda s: s.name)
@pytest.mark.parametrize("style", [0, 1])
def test_query_finish_is_norm_then_rotation(shape, style):
    from kvd_synth import with_style
    shape = with_style(shape, style)
    ctx, _ = open_layer(shape, max_tokens=4096)
    rng = np.random.Generator(np.random.PCG64(9))
    m, nq, dh = 7, shape.n_q_heads, shape.d_head
    stride = nq * dh + 64
    Q, Gq = _bits(rng, (m, stride), 1.5), _bits(rng, (dh,), 0.1, 1.0)
    pos = np.array([0, 1, 15, 16, 1000, 4095, 77], dtype=np.int32)
    out = torch.empty((m, nq, dh), dtype=torch.bfloat16, device="cuda")
    gq = dev(Gq) if shape.qk_norm else None
    ctx.kvd_scaffold_query_finish(0, dev(Q), stride, torch.from_numpy(pos).cuda(), m, gq, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    q = bf16_to_f64(Q)
    ref = np.empty((m, nq, dh))
    for r in range(m):
        for h in range(nq):
            v = q[r, h * dh:(h + 1) * dh]
            if shape.qk_norm:
                v = oracle.rmsnorm(v, bf16_to_f64(Gq), shape.rms_eps)
            ref[r, h] = oracle.rope(v, int(pos[r]), shape.rope_theta, style)
    got = host_f64(out)
    assert np.max(np.abs(got - ref)) <= 2 ** -8 * np.max(np.abs(ref)) + 1e-6
    assert np.linalg.norm(got - ref) <= 4e-3 * np.linalg.norm(ref)
    ctx.close()


def test_elementwise_steps_and_greedy_pick():
    shape = GEMMA3_4B_GLOBAL
    ctx, _ = open_layer(shape, max_tokens=256)
    rng = np.random.Generator(np.random.PCG64(3))
    m, d, width = 9, 2560, 1280
    # residual add
    H, Y = _bits(rng, (m, d), 1.0), _bits(rng, (m, d + 256), 1.0)
    h = dev(H)
    ctx.kvd_scaffold_add_rows(h, dev(Y), d + 256, m, d)
    want = f32_to_bf16_bits((bf16_to_f64(H) + bf16_to_f64(Y)[:, :d]).astype(np.float32))
    assert np.array_equal(host_bits(h), want)  # one rounded fp32 addition: exact
    # gated activation, both kinds
    GU = _bits(rng, (m, 2 * width + 128), 2.0)
    g, u = bf16_to_f64(GU)[:, :width], bf16_to_f64(GU)[:, width:2 * width]
    for act, f in ((KVD_ACT_SILU, lambda x: x / (1.0 + np.exp(-x))),
                   (KVD_ACT_GELU_TANH, lambda x: 0.5 * x * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x ** 3))))):
        out = torch.empty((m, width), dtype=torch.bfloat16, device="cuda")
        ctx.kvd_scaffold_gated_act(dev(GU), 2 * width + 128, m, width, act, out)
        ref = f(g) * u
        assert np.max(np.abs(host_f64(out) - ref)) <= 2 ** -8 * np.max(np.abs(ref)) + 1e-6
    # embedding gather
    table = _bits(rng, (50, d), 1.0)
    toks = np.array([3, 49, 0, 3], dtype=np.int32)
    e = torch.empty((4, d), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_scaffold_embed(dev(table), torch.from_numpy(toks).cuda(), 4, d, 50, e)
    assert np.array_equal(host_bits(e), table[toks])
    # greedy pick: the lowest index among equal maxima; padding columns are not looked at
    L = _bits(rng, (3, 1000 + 24), 1.0)
    L[0, 700] = L[0, 123] = 0x4120  # 10.0 twice
    L[1, 999] = 0x4120
    L[2, :1000] = 0x3F80             # all equal
    L[:, 1000:] = 0x4220             # 40.0 in the padding
    t = torch.empty((3,), dtype=torch.int32, device="cuda")
    ctx.kvd_scaffold_argmax(dev(L), 1024, 3, 1000, t)
    assert t.tolist() == [123, 999, 0]
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    ctx.close()
