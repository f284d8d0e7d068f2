"""FP4 residual checkpoints on the GPU (kvd_checkpoint_residual_fp4 / kvd_recompute_kv_fp4) against their oracle.

  * what the quantising checkpoint stores -- E2M1 codes, E4M3 block scales, power-of-two row scales, positions and
    the sum of squares of the ORIGINAL row -- equals the oracle's quantisation EXACTLY (an encoding decided in fp32
    on both sides; the statistic has the bits the bf16 store keeps);
  * K/V recomputed from the FP4 store follow the FP4 oracle (relative Frobenius 1e-2 as for the bf16 path; max abs
    1e-2 plus the bf16 output's half-ulp at the largest magnitude) on Gemma-, Qwen- and SmolLM-shaped layers, several
    ranges and sequences in one call;
  * a row's K/V bits do not depend on the ranges it is recomputed with;
  * the distance to the UNQUANTISED definition is reported and loosely bounded (the format's accuracy, not a claim);
  * sizes, limits and the memory report.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from oracle import fp4, fp8
from kvd_synth import GEMMA3_4B_GLOBAL, QWEN3_4B, SMOLLM2_135M, bf16_to_f64, make_residuals
from gpu_util import dev, host_f64, kv_errors, open_layer, oracle_kv

pytestmark = pytest.mark.gpu

E2M1 = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6, -0.0, -0.5, -1, -1.5, -2, -3, -4, -6])


def open_fp4(shape, max_tokens, max_seqs=1):
    ctx, w = open_layer(shape, max_tokens=max_tokens, max_seqs=max_seqs, max_batch=max_seqs)
    arena = torch.zeros(kvd.kvd_store_bytes_fp4(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp4(arena, 1)
    return ctx, w, arena


def regions(arena, slots, d):
    """The five regions of a one-layer FP4 arena as host arrays."""
    ru = lambda x: (x + 255) // 256 * 256
    a = arena.cpu().numpy()
    o = 0
    codes = a[o:o + slots * d // 2].reshape(slots, d // 2)
    o += ru(slots * d // 2)
    block = a[o:o + slots * d // 16].reshape(slots, d // 16)
    o += ru(slots * d // 16)
    pos = a[o:o + slots * 4].view(np.int32)
    o += ru(slots * 4)
    sumsq = a[o:o + slots * 4].view(np.float32)
    o += ru(slots * 4)
    scale = a[o:o + slots * 4].view(np.float32)
    return codes, block, pos, sumsq, scale


def oracle_args(shape, w):
    return (bf16_to_f64(w.gamma_in), bf16_to_f64(w.w_kv), shape.n_kv_heads, shape.d_head, shape.rms_eps, shape.rope_theta,
            bf16_to_f64(w.gamma_k) if w.gamma_k is not None else None, shape.rms_eps, shape.rope_style)


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, SMOLLM2_135M], ids=lambda s: s.name)
def test_stored_codes_scales_and_statistics_equal_the_oracles_quantisation(shape):
    n, d, max_tokens = 203, shape.d_hidden, 256
    ctx, w, arena = open_fp4(shape, max_tokens)
    X = make_residuals(shape, n, seed=51, outliers=True)
    X[7] = 0            # an all-zero row
    X[9, 16:32] = 0     # an all-zero block
    pos = np.arange(n) * 3 + 1
    ctx.kvd_checkpoint_residual_fp4(0, 0, dev(X), torch.from_numpy(pos.astype(np.int32)).cuda(), n)
    assert ctx.kvd_poll_status() == kvd.KVD_OK and ctx.kvd_rows_stored_fp4(0, 0) == n
    codes, block, spos, sumsq, scale = regions(arena, max_tokens, d)
    want_codes, want_block, want_row = fp4.quantize_rows_fp4(bf16_to_f64(X))
    got_codes = np.empty((n, d))
    got_codes[:, 0::2] = E2M1[codes[:n] & 0xF]
    got_codes[:, 1::2] = E2M1[codes[:n] >> 4]
    assert np.array_equal(np.abs(got_codes), np.abs(want_codes)) and np.array_equal(got_codes < 0, (want_codes < 0))
    got_block = torch.from_numpy(block[:n].copy()).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    assert np.array_equal(got_block, want_block)
    assert np.array_equal(scale[:n].astype(np.float64), want_row)
    assert np.array_equal(spos[:n], pos)
    # the statistic is the ORIGINAL row's, with the bits the bf16 checkpoint stores
    ctx2, _ = open_layer(shape, max_tokens=max_tokens, with_store=True)
    ctx2.kvd_checkpoint_residual(0, 0, dev(X), torch.from_numpy(pos.astype(np.int32)).cuda(), n)
    a2 = ctx2._keep[-1].cpu().numpy()
    ru = lambda x: (x + 255) // 256 * 256
    ss2 = a2[ru(max_tokens * d * 2) + ru(max_tokens * 4):][:max_tokens * 4].view(np.float32)
    assert np.array_equal(sumsq[:n].view(np.uint32), ss2[:n].view(np.uint32))
    # untouched slots stay zero
    assert not codes[n:].any() and not block[n:].any()
    ctx.close()
    ctx2.close()


@pytest.mark.parametrize("shape,n", [(GEMMA3_4B_GLOBAL, 700), (QWEN3_4B, 300), (SMOLLM2_135M, 130)], ids=lambda v: getattr(v, "name", v))
def test_recompute_from_fp4_checkpoints_follows_the_fp4_oracle(shape, n):
    ctx, w, _ = open_fp4(shape, 1024, max_seqs=2)
    kdim = shape.n_kv_heads * shape.d_head
    X = make_residuals(shape, n, seed=52, outliers=shape is GEMMA3_4B_GLOBAL)
    pos = np.arange(n) + 5
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    ctx.kvd_checkpoint_residual_fp4(0, 0, x, p, n)
    ctx.kvd_checkpoint_residual_fp4(1, 0, x[: n // 2], p[: n // 2], n // 2)
    a, b = n // 3, n - n // 3 - 1  # two ranges of sequence 0 and one of sequence 1, ragged against the 256-row blocks
    scratch = torch.empty(kvd.kvd_fp4_scratch_bytes(ctx.desc, a + b + n // 2), dtype=torch.uint8, device="cuda")
    k = [torch.full((m + 1, kdim), 5.0, dtype=torch.bfloat16, device="cuda") for m in (a, b, n // 2)]
    v = [torch.full_like(t, 5.0) for t in k]
    n0 = ctx.kvd_launch_count()
    ctx.kvd_recompute_kv_fp4(0, [(0, 0, a, k[0], v[0]), (0, a + 1, b, k[1], v[1]), (1, 0, n // 2, k[2], v[2])], kdim, scratch)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert ctx.kvd_launch_count() - n0 == 2  # expand + projection
    Kr, Vr = fp4.recompute_kv_fp4(bf16_to_f64(X), pos, *oracle_args(shape, w))
    Kp, Vp = oracle_kv(shape, w, X, pos)   # the unquantised definition, for the accuracy report
    for (t_k, t_v, rows) in ((k[0], v[0], slice(0, a)), (k[1], v[1], slice(a + 1, a + 1 + b)), (k[2], v[2], slice(0, n // 2))):
        m = rows.stop - rows.start
        assert torch.all(t_k[m:] == 5.0) and torch.all(t_v[m:] == 5.0)  # nothing written past the range
        for name, g, r, plain in (("K", host_f64(t_k[:m]), Kr[rows].reshape(m, kdim), Kp[rows].reshape(m, kdim)),
                                  ("V", host_f64(t_v[:m]), Vr[rows].reshape(m, kdim), Vp[rows].reshape(m, kdim))):
            mx, rel = kv_errors(g, r)
            # absolute bound: 1e-2 for the arithmetic (fp32 accumulation, the bf16 rounding of the folded weights) plus
            # the bf16 output's own half-ulp at the largest magnitude (rows decoded from 4-bit codes spread V a little
            # wider than bf16 rows do: |V| passes 4 here, where that half-ulp alone is 0.0156)
            assert mx <= 1e-2 + 2.0 ** -8 * np.max(np.abs(r)) and rel <= 1e-2, (name, mx, rel, np.max(np.abs(r)))
            far = np.linalg.norm(g - plain) / np.linalg.norm(plain)
            assert far < 0.35, (name, far)  # the format's distance from the unquantised K/V: reported below
    print(f"{shape.name}: K/V from FP4 rows vs the unquantised definition: relative Frobenius "
          f"{np.linalg.norm(host_f64(k[0][:a]) - Kp[:a].reshape(a, kdim)) / np.linalg.norm(Kp[:a]):.3f} (K), "
          f"{np.linalg.norm(host_f64(v[0][:a]) - Vp[:a].reshape(a, kdim)) / np.linalg.norm(Vp[:a]):.3f} (V)")
    # a row's bits do not depend on the ranges it is recomputed with
    one_k, one_v = torch.zeros((1, kdim), dtype=torch.bfloat16, device="cuda"), torch.zeros((1, kdim), dtype=torch.bfloat16, device="cuda")
    for r in (0, a - 1, a + 1, n - 1):
        ctx.kvd_recompute_kv_fp4(0, [(0, r, 1, one_k, one_v)], kdim, scratch)
        src_k, src_v, idx = (k[0], v[0], r) if r < a else (k[1], v[1], r - a - 1)
        assert torch.equal(one_k[0], src_k[idx]) and torch.equal(one_v[0], src_v[idx]), r
    ctx.close()


def test_fp4_sizes_limits_and_memory_report():
    shape = GEMMA3_4B_GLOBAL
    ctx, _, _ = open_fp4(shape, 64)
    d = shape.d_hidden
    assert kvd.kvd_store_bytes_fp4(ctx.desc, 1) == 64 * (d // 2 + d // 16 + 12)
    assert kvd.kvd_fp4_scratch_bytes(ctx.desc, 10) >= 10 * (2 * d + 8)
    kdim = shape.n_kv_heads * shape.d_head
    x = dev(make_residuals(shape, 64, seed=1))
    p = torch.arange(64, dtype=torch.int32, device="cuda")
    ctx.kvd_checkpoint_residual_fp4(0, 0, x, p, 60)
    assert ctx.kvd_memory_stats()["checkpoint_bytes_used"] == 60 * (d // 2 + d // 16 + 12)
    with pytest.raises(kvd.KvdError) as e:   # the sequence's slab is full
        ctx.kvd_checkpoint_residual_fp4(0, 0, x, p, 5)
    assert e.value.status == 4
    k = torch.zeros((64, kdim), dtype=torch.bfloat16, device="cuda")
    small = torch.empty(kvd.kvd_fp4_scratch_bytes(ctx.desc, 10), dtype=torch.uint8, device="cuda")
    for ranges, status in (([(0, 0, 61, k, k)], 4), ([(0, 0, 60, k, k)], 4), ([(1, 0, 1, k, k)], 1)):
        with pytest.raises(kvd.KvdError) as e:  # more rows than stored; a scratch that is too small; a bad slot
            ctx.kvd_recompute_kv_fp4(0, ranges, kdim, small)
        assert e.value.status == status, ranges
    ctx.kvd_reset_sequence_fp4(0)
    assert ctx.kvd_rows_stored_fp4(0, 0) == 0
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    ctx.close()
