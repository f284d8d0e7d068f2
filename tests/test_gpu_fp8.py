"""GPU parity of the FP8 checkpoint variant (kvd_checkpoint_residual_fp8 / kvd_recompute_kv_fp8) through the C ABI.

  * the stored codes, scales, sums of squares and positions equal the oracle's quantisation exactly (the
    codes are an encoding decided in fp32 on both sides);
  * K/V recomputed from the FP8 store follow oracle.fp8.recompute_kv_fp8 with the tolerance of the bf16
    path (max abs 2e-2, rel Frobenius 1e-2): the quantisation is part of the definition, not of the error;
  * against the unquantised result the variant is a few per cent off (reported, bounded);
  * a row's bits do not depend on the batch it is recomputed in.
"""
import numpy as np
import pytest
import torch

import paper_2603_19664_b200 as kvd
from kvd_synth import GEMMA3_4B_GLOBAL, QWEN3_4B, SMOLLM2_135M, bf16_to_f64, make_residuals
from gpu_util import dev, host_bits, host_f64, kv_errors, open_layer, oracle_kv
from oracle import fp8 as ofp8
from test_oracle_fp8 import decode_e4m3

pytestmark = pytest.mark.gpu

LUT = np.array([decode_e4m3(c) for c in range(256)])


def open_fp8(shape, max_tokens, max_seqs=1):
    ctx, w = open_layer(shape, max_tokens=max_tokens, max_seqs=max_seqs)
    arena = torch.zeros(kvd.kvd_store_bytes_fp8(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena, 1)
    return ctx, w, arena


def oracle_fp8_kv(shape, w, X_bits, pos):
    return ofp8.recompute_kv_fp8(bf16_to_f64(X_bits), np.asarray(pos, np.int32), bf16_to_f64(w.gamma_in),
                                 bf16_to_f64(w.w_kv), shape.n_kv_heads, shape.d_head, shape.rms_eps, shape.rope_theta,
                                 bf16_to_f64(w.gamma_k) if w.gamma_k is not None else None, shape.rms_eps,
                                 shape.rope_style)


def test_stored_codes_scales_and_statistics_equal_the_oracles_quantisation():
    shape = GEMMA3_4B_GLOBAL
    max_tokens, n = 384, 300
    ctx, w, arena = open_fp8(shape, max_tokens, max_seqs=2)
    X = make_residuals(shape, n, seed=31, outliers=True)
    pos = np.arange(n) + 9
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    ctx.kvd_checkpoint_residual_fp8(1, 0, x[:11], p[:11], 11)
    ctx.kvd_checkpoint_residual_fp8(1, 0, x[11:], p[11:], n - 11)
    torch.cuda.synchronize()
    assert ctx.kvd_rows_stored_fp8(0, 1) == n and ctx.kvd_rows_stored_fp8(0, 0) == 0
    assert ctx.kvd_memory_stats()["checkpoint_bytes_used"] == n * (shape.d_hidden + 12)
    slots = 2 * max_tokens
    ru = lambda b: (b + 255) // 256 * 256
    c_bytes, f_bytes = ru(slots * shape.d_hidden), ru(slots * 4)
    assert arena.numel() == c_bytes + 3 * f_bytes
    a = arena.cpu().numpy()
    codes = a[:c_bytes].reshape(-1, shape.d_hidden)[max_tokens:max_tokens + n]
    got_pos = a[c_bytes:c_bytes + f_bytes].view(np.int32)[max_tokens:max_tokens + n]
    got_ss = a[c_bytes + f_bytes:c_bytes + 2 * f_bytes].view(np.float32)[max_tokens:max_tokens + n]
    got_sc = a[c_bytes + 2 * f_bytes:].view(np.float32)[max_tokens:max_tokens + n]
    Xf = bf16_to_f64(X)
    q, s = ofp8.quantize_rows(Xf)
    assert np.array_equal(got_sc.astype(np.float64), s)
    assert np.array_equal(LUT[codes], q)            # every code decodes to the oracle's grid value
    assert np.array_equal(got_pos, pos)
    ref = np.sum(Xf ** 2, axis=1)
    assert np.max(np.abs(got_ss - ref) / ref) < 1e-6
    # the statistic has the bits the bf16 store keeps for the same rows (one function takes it everywhere)
    arena16 = torch.zeros(kvd.kvd_store_bytes(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store(arena16, 1)
    ctx.kvd_checkpoint_residual(1, 0, x, p, n)
    torch.cuda.synchronize()
    a16 = arena16.cpu().numpy()
    r_bytes = ru(slots * shape.d_hidden * 2)
    ss16 = a16[r_bytes + f_bytes:].view(np.float32)[max_tokens:max_tokens + n]
    assert np.array_equal(ss16.view(np.uint32), got_ss.view(np.uint32))


@pytest.mark.parametrize("shape,n", [(GEMMA3_4B_GLOBAL, 300), (GEMMA3_4B_GLOBAL, 1), (QWEN3_4B, 700), (SMOLLM2_135M, 130)],
                         ids=lambda v: getattr(v, "name", v))
def test_recompute_from_fp8_checkpoints_follows_the_fp8_oracle(shape, n):
    ctx, w, arena = open_fp8(shape, 1024)
    kdim = shape.n_kv_heads * shape.d_head
    X = make_residuals(shape, n, seed=32, outliers=True)
    pos = np.arange(n) + 40
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    ctx.kvd_checkpoint_residual_fp8(0, 0, x, p, n)
    k = torch.full((n + 2, kdim), -7.0, dtype=torch.bfloat16, device="cuda")
    v = torch.full_like(k, -7.0)
    ctx.kvd_recompute_kv_fp8(0, [(0, 0, n, k, v)], kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.all(k[n:] == -7.0) and torch.all(v[n:] == -7.0)   # guard rows untouched
    Kr, Vr = oracle_fp8_kv(shape, w, X, pos)
    for name, g, r in (("K", host_f64(k)[:n], Kr.reshape(n, kdim)), ("V", host_f64(v)[:n], Vr.reshape(n, kdim))):
        mx, rel = kv_errors(g, r)
        assert mx <= 2e-2 and rel <= 1e-2, (name, mx, rel)
    # against the unquantised definition: a few per cent of the rms, as the format predicts
    Ke, Ve = oracle_kv(shape, w, X, pos)
    for name, g, r in (("K", host_f64(k)[:n], Ke.reshape(n, kdim)), ("V", host_f64(v)[:n], Ve.reshape(n, kdim))):
        rel = np.linalg.norm(g - r) / np.linalg.norm(r)
        assert rel < 0.08, (name, rel)


def test_fp8_recompute_at_the_bench_size_sampled_against_the_fp8_oracle():
    """T = 4096 rows of the Gemma-3-4B-shaped layer (the configuration bench.py times), a seeded sample of rows
    plus the first and last row of every 128-row block class against the FP8 oracle."""
    shape = GEMMA3_4B_GLOBAL
    T = 4096
    ctx, w, arena = open_fp8(shape, T + 8)
    kdim = shape.n_kv_heads * shape.d_head
    X = make_residuals(shape, T, seed=34, outliers=True)
    pos = np.arange(T)
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    ctx.kvd_checkpoint_residual_fp8(0, 0, x, p, T)
    k = torch.zeros((T, kdim), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros_like(k)
    ctx.kvd_recompute_kv_fp8(0, [(0, 0, T, k, v)], kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    rows = np.unique(np.concatenate([np.random.default_rng(5).choice(T, 512, replace=False),
                                     [0, 127, 128, 255, 256, 2047, 2048, T - 129, T - 128, T - 1]]))
    Kr, Vr = oracle_fp8_kv(shape, w, X[rows], pos[rows])
    for name, g, r in (("K", host_f64(k)[rows], Kr.reshape(len(rows), kdim)), ("V", host_f64(v)[rows], Vr.reshape(len(rows), kdim))):
        mx, rel = kv_errors(g, r)
        assert mx <= 2e-2 and rel <= 1e-2, (name, mx, rel)


def test_fp8_recompute_bits_do_not_depend_on_the_batch():
    shape = GEMMA3_4B_GLOBAL
    ctx, w, arena = open_fp8(shape, 2048, max_seqs=2)
    kdim = shape.n_kv_heads * shape.d_head
    T = 1100
    X = make_residuals(shape, T, seed=33, outliers=True)
    pos = np.arange(T)
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    ctx.kvd_checkpoint_residual_fp8(0, 0, x, p, T)
    ctx.kvd_checkpoint_residual_fp8(1, 0, x[500:], p[500:], T - 500)   # the same rows again in another slot
    K = torch.zeros((T, kdim), dtype=torch.bfloat16, device="cuda")
    V = torch.zeros_like(K)
    ctx.kvd_recompute_kv_fp8(0, [(0, 0, T, K, V)], kdim)
    Kb, Vb = host_bits(K), host_bits(V)
    for seq, first, n, src0 in ((0, 0, 1, 0), (0, 255, 3, 255), (0, 700, 257, 700), (1, 0, 600, 500), (1, 100, 129, 600)):
        k = torch.zeros((n, kdim), dtype=torch.bfloat16, device="cuda")
        v = torch.zeros_like(k)
        ctx.kvd_recompute_kv_fp8(0, [(seq, first, n, k, v)], kdim)
        assert np.array_equal(host_bits(k), Kb[src0:src0 + n]) and np.array_equal(host_bits(v), Vb[src0:src0 + n])
    # two ranges in one launch
    k1 = torch.zeros((300, kdim), dtype=torch.bfloat16, device="cuda"); v1 = torch.zeros_like(k1)
    k2 = torch.zeros((40, kdim), dtype=torch.bfloat16, device="cuda"); v2 = torch.zeros_like(k2)
    ctx.kvd_recompute_kv_fp8(0, [(0, 10, 300, k1, v1), (1, 0, 40, k2, v2)], kdim)
    assert np.array_equal(host_bits(k1), Kb[10:310]) and np.array_equal(host_bits(v2), Vb[500:540])
    assert ctx.kvd_poll_status() == kvd.KVD_OK


def test_fp8_argument_errors():
    shape = GEMMA3_4B_GLOBAL
    ctx, w = open_layer(shape, max_tokens=256)
    kdim = shape.n_kv_heads * shape.d_head
    k = torch.zeros((8, kdim), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(kvd.KvdError) as e:          # no FP8 store attached
        ctx.kvd_recompute_kv_fp8(0, [(0, 0, 8, k, k)], kdim)
    assert e.value.status == 5
    arena = torch.zeros(kvd.kvd_store_bytes_fp8(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena, 1)
    with pytest.raises(kvd.KvdError) as e:          # more rows than stored
        ctx.kvd_recompute_kv_fp8(0, [(0, 0, 8, k, k)], kdim)
    assert e.value.status == 4
    assert ctx.kvd_poll_status() == kvd.KVD_OK


def test_caller_held_quantised_rows_give_the_bits_of_rows_in_the_store():
    """kvd_quantize_rows_fp8 + the _rows forms: the new tokens of a batch in one contiguous caller buffer instead
    of one store range per sequence.  Codes, scales and statistics equal what the checkpoint stores; K/V from the
    caller's rows equal K/V from the same rows in the store, alone and next to store ranges in one launch."""
    shape = GEMMA3_4B_GLOBAL
    ctx, w, arena = open_fp8(shape, 512, max_seqs=2)
    kdim = shape.n_kv_heads * shape.d_head
    n = 70
    X = make_residuals(shape, n, seed=35, outliers=True)
    pos = np.arange(n) + 100
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    ctx.kvd_checkpoint_residual_fp8(0, 0, x, p, n)
    codes = torch.zeros((n, shape.d_hidden), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((n,), dtype=torch.float32, device="cuda")
    sumsq = torch.zeros_like(scales)
    ctx.kvd_quantize_rows_fp8(x, n, codes, scales, sumsq)
    torch.cuda.synchronize()
    q_ref, s_ref = ofp8.quantize_rows(bf16_to_f64(X))
    assert np.array_equal(LUT[codes.cpu().numpy()], q_ref) and np.array_equal(scales.cpu().numpy().astype(np.float64), s_ref)
    a = arena.cpu().numpy()
    ru = lambda b: (b + 255) // 256 * 256
    slots = 2 * 512
    c_bytes, f_bytes = ru(slots * shape.d_hidden), ru(slots * 4)
    assert np.array_equal(a[:c_bytes].reshape(-1, shape.d_hidden)[:n], codes.cpu().numpy())
    assert np.array_equal(a[c_bytes + f_bytes:c_bytes + 2 * f_bytes].view(np.uint32)[:n], sumsq.cpu().numpy().view(np.uint32))
    # K/V: from the store, from the caller's rows, and both kinds of source in one launch
    ks = torch.zeros((n, kdim), dtype=torch.bfloat16, device="cuda"); vs = torch.zeros_like(ks)
    kc = torch.zeros_like(ks); vc = torch.zeros_like(ks)
    ctx.kvd_recompute_kv_fp8(0, [(0, 0, n, ks, vs)], kdim)
    ctx.kvd_recompute_kv_fp8_rows(0, [], (codes, scales, sumsq, p, n, kc, vc), kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.equal(ks, kc) and torch.equal(vs, vc) and float(kc.abs().max()) > 0
    k1 = torch.zeros((40, kdim), dtype=torch.bfloat16, device="cuda"); v1 = torch.zeros_like(k1)
    k2 = torch.zeros((3, kdim), dtype=torch.bfloat16, device="cuda"); v2 = torch.zeros_like(k2)
    ctx.kvd_recompute_kv_fp8_rows(0, [(0, 5, 40, k1, v1)], (codes[60:], scales[60:], sumsq[60:], p[60:], 3, k2, v2), kdim)
    assert torch.equal(k1, ks[5:45]) and torch.equal(v1, vs[5:45]) and torch.equal(k2, ks[60:63]) and torch.equal(v2, vs[60:63])
    with pytest.raises(kvd.KvdError) as e:      # incomplete description of the rows
        ctx.kvd_recompute_kv_fp8_rows(0, [], (codes, None, sumsq, p, n, kc, vc), kdim)
    assert e.value.status == 1
    assert ctx.kvd_poll_status() == kvd.KVD_OK
