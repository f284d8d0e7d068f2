"""The recompute path with fp32 rows, weights and outputs (kvd_set_dtype(2)): the "float32" regime of the
paper's Section 5.1 check.  The tensor cores read the fp32 operands as TF32 (10-bit mantissa) and accumulate
in fp32, so against the fp64 oracle on the same fp32 inputs the error is that of TF32 products (about 1e-3
relative) -- inside the K/V tolerance; what the section asserts, and what is checked bit for bit, is that
K/V rebuilt from checkpointed rows equal the K/V of the first pass at every length 16 ... 256.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from kvd_synth import GEMMA3_4B_GLOBAL, QWEN3_4B, SMOLLM2_135M, bf16_to_f64, make_layer_weights, make_residuals

pytestmark = pytest.mark.gpu


def f32(bits_bf16: np.ndarray, seed: int) -> np.ndarray:
    """The synthetic bf16-valued array with low-order fp32 bits added (so that the inputs are not TF32-exact)."""
    a = bf16_to_f64(bits_bf16)
    noise = np.random.default_rng(seed).uniform(-1.0, 1.0, size=a.shape) * 2.0 ** -12
    return (a * (1.0 + noise)).astype(np.float32)


def open_f32(shape, max_tokens):
    w = make_layer_weights(shape)
    desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                         shape.qk_norm, shape.rms_eps, shape.rope_style, 1, max_tokens, 1)
    ctx = kvd.Kvd(desc)
    ctx.kvd_set_dtype(2)
    w32 = {"w_kv": f32(w.w_kv, 1), "gamma_in": f32(w.gamma_in, 2),
           "gamma_k": f32(w.gamma_k, 3) if w.gamma_k is not None else None}
    t = {k: (torch.from_numpy(v).cuda() if v is not None else None) for k, v in w32.items()}
    ctx.kvd_set_layer(0, t["w_kv"], t["gamma_in"], t["gamma_k"], shape.rope_theta, shape.sliding_window)
    arena = torch.zeros(kvd.kvd_store_bytes_dtype(desc, 1, 2), dtype=torch.uint8, device="cuda")
    assert arena.numel() > kvd.kvd_store_bytes(desc, 1)
    ctx.kvd_attach_store(arena, 1)
    return ctx, w32


@pytest.mark.parametrize("shape,n", [(GEMMA3_4B_GLOBAL, 300), (QWEN3_4B, 130), (SMOLLM2_135M, 200), (GEMMA3_4B_GLOBAL, 1)],
                         ids=lambda v: getattr(v, "name", v))
def test_fp32_recompute_follows_the_oracle(shape, n):
    ctx, w32 = open_f32(shape, 1024)
    kdim = shape.n_kv_heads * shape.d_head
    X32 = f32(make_residuals(shape, n, seed=41, outliers=True), 4)
    pos = np.arange(n) + 17
    x, p = torch.from_numpy(X32).cuda(), torch.from_numpy(pos.astype(np.int32)).cuda()
    k = torch.full((n + 1, kdim), -7.0, dtype=torch.float32, device="cuda")
    v = torch.full_like(k, -7.0)
    ctx.kvd_recompute_kv(0, x, p, n, k, v, kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.all(k[n:] == -7.0) and torch.all(v[n:] == -7.0)
    f = lambda a: None if a is None else a.astype(np.float64)
    Kr, Vr = oracle.recompute_kv(f(X32), pos.astype(np.int32), f(w32["gamma_in"]), f(w32["w_kv"]), shape.n_kv_heads,
                                 shape.d_head, shape.rms_eps, shape.rope_theta, f(w32["gamma_k"]), shape.rms_eps,
                                 shape.rope_style)
    for name, g, r in (("K", k[:n].cpu().numpy().astype(np.float64), Kr.reshape(n, kdim)),
                       ("V", v[:n].cpu().numpy().astype(np.float64), Vr.reshape(n, kdim))):
        d = g - r
        assert np.max(np.abs(d)) <= 2e-2, name
        rel = np.linalg.norm(d) / np.linalg.norm(r)
        assert rel <= 2e-3, (name, rel)          # TF32 operands: 2^-11 per factor


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, SMOLLM2_135M], ids=lambda s: s.name)
def test_fp32_reconstruction_is_bit_exact_at_every_length(shape):
    ctx, w32 = open_f32(shape, 512)
    kdim = shape.n_kv_heads * shape.d_head
    for length in (16, 32, 64, 128, 256):
        X32 = f32(make_residuals(shape, length, seed=50 + length, outliers=True), 5)
        x, p = torch.from_numpy(X32).cuda(), torch.arange(length, dtype=torch.int32, device="cuda")
        kc = torch.zeros((length, kdim), dtype=torch.float32, device="cuda")
        vc = torch.zeros_like(kc)
        h = length // 2
        ctx.kvd_recompute_kv(0, x[:h], p[:h], h, kc[:h], vc[:h], kdim)
        for m in range(h, length):
            ctx.kvd_recompute_kv(0, x[m:m + 1], p[m:m + 1], 1, kc[m:m + 1], vc[m:m + 1], kdim)
        ctx.kvd_reset_sequence(0)
        ctx.kvd_checkpoint_residual(0, 0, x, p, length)
        kr = torch.zeros_like(kc)
        vr = torch.zeros_like(vc)
        ctx.kvd_recompute_kv(0, None, None, length, kr, vr, kdim, seq=0, first_row=0)
        assert ctx.kvd_poll_status() == kvd.KVD_OK
        assert torch.equal(kr.view(torch.int32), kc.view(torch.int32)), length
        assert torch.equal(vr.view(torch.int32), vc.view(torch.int32)), length
        assert float(kr.abs().max()) > 0


def test_fp32_context_has_no_attention_and_its_store_is_twice_as_large():
    shape = GEMMA3_4B_GLOBAL
    ctx, w32 = open_f32(shape, 256)
    assert kvd.kvd_store_bytes_dtype(ctx.desc, 1, 2) == 256 * shape.d_hidden * 4 + 2 * 256 * 4
    assert kvd.kvd_store_bytes_dtype(ctx.desc, 1, 7) == 0
    ws = torch.empty(kvd.kvd_workspace_bytes(ctx.desc), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_workspace(ws)
    kdim = shape.n_kv_heads * shape.d_head
    q = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.float32, device="cuda")
    k = torch.zeros((4, kdim), dtype=torch.float32, device="cuda")
    with pytest.raises(kvd.KvdError) as e:
        ctx.kvd_decode_attention(0, 1, q, [3], [[(k, k, kdim, 0, 4)]], 0.0, q)
    assert e.value.status == 6
    x = torch.zeros((3, shape.d_hidden), dtype=torch.float32, device="cuda")
    ctx.kvd_checkpoint_residual(0, 0, x, torch.arange(3, dtype=torch.int32, device="cuda"), 3)
    assert ctx.kvd_memory_stats()["checkpoint_bytes_used"] == 3 * (shape.d_hidden * 4 + 8)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
