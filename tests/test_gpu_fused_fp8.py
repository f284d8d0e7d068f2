"""GPU parity of kvd_decode_attention_recompute_fp8 (FP8 checkpoints rebuilt and attended in one kernel).

The call must give attention over [K/V rebuilt from ranges of the FP8 store] + [live segments]:
  * against the fp64 oracle of the FP8 variant (oracle.fp8.recompute_kv_fp8 for every key, then
    oracle.decode_attention), with the attention tolerance: rel Frobenius <= 1e-2, max abs <= 1e-2 max |oracle|;
  * against the two-call GPU path (kvd_recompute_kv_fp8 + kvd_decode_attention), equal up to rounding;
  * the K/V of the ranges that are stored (the new tokens) have the bits kvd_recompute_kv_fp8 gives.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from kvd_synth import GEMMA3_4B_GLOBAL, GEMMA3_4B_LOCAL, QWEN3_4B, SMOLLM2_135M, bf16_to_f64, make_query, make_residuals
from gpu_util import dev, host_f64, open_layer
from test_gpu_fused import attn_check
from test_gpu_fp8 import oracle_fp8_kv

pytestmark = pytest.mark.gpu


def run_case(shape, n_old_list, n_live, pos0_list=None, max_tokens=4096, seed=1, keep_nothing=False):
    """One decode step of a batch; every row of sequence b (n_old evicted, n_live live, the current token) is in
    the FP8 store.  keep_nothing: no live segments at all -- the range covers every token, the current one too.
    Returns (fused out, two-call out, oracle out)."""
    batch = len(n_old_list)
    ctx, w = open_layer(shape, max_tokens=max_tokens, max_batch=batch, max_seqs=batch)
    arena = torch.zeros(kvd.kvd_store_bytes_fp8(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena, 1)
    kdim = shape.n_kv_heads * shape.d_head
    pos0_list = pos0_list or [0] * batch
    q_bits = make_query(shape, batch, seed=seed)
    q = dev(q_bits)
    X_all, pos_all, q_pos, bufs = [], [], [], []
    for b in range(batch):
        T = n_old_list[b] + n_live + 1
        X = make_residuals(shape, T, seed=seed * 100 + b, outliers=True)
        pos = np.arange(T) + pos0_list[b]
        X_all.append(X)
        pos_all.append(pos)
        ctx.kvd_checkpoint_residual_fp8(b, 0, dev(X), torch.from_numpy(pos.astype(np.int32)).cuda(), T)
        q_pos.append(int(pos[T - 1]))
        k = torch.zeros((T, kdim), dtype=torch.bfloat16, device="cuda")   # row i = K of token i where it is stored
        bufs.append((k, torch.zeros_like(k)))
        if n_live and not keep_nothing:
            n_old = n_old_list[b]
            ctx.kvd_recompute_kv_fp8(0, [(b, n_old, n_live, k[n_old:], bufs[b][1][n_old:])], kdim)

    def live_segs():
        out = []
        for b in range(batch):
            n_old, T = n_old_list[b], n_old_list[b] + n_live + 1
            k, v = bufs[b]
            row = []
            if not keep_nothing:
                if n_live:
                    row.append((k[n_old:], v[n_old:], kdim, pos0_list[b] + n_old, n_live))
                row.append((k[T - 1:], v[T - 1:], kdim, q_pos[b], 1))
            out.append(row)
        return out

    out_f = torch.full((batch, shape.n_q_heads, shape.d_head), 9.0, dtype=torch.bfloat16, device="cuda")
    if keep_nothing:
        ranges = [(b, 0, n_old_list[b] + n_live + 1) for b in range(batch)]
        stores = []
    else:
        ranges = [(b, 0, n_old_list[b]) for b in range(batch)]
        stores = [(b, n_old_list[b] + n_live, 1, bufs[b][0][n_old_list[b] + n_live:], bufs[b][1][n_old_list[b] + n_live:])
                  for b in range(batch)]
    ctx.kvd_decode_attention_recompute_fp8(0, batch, q, q_pos, ranges, stores, kdim, live_segs(), 0.0, out_f)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    cur_fused = [(bufs[b][0][-1].clone(), bufs[b][1][-1].clone()) for b in range(batch)]
    # the two-call path: everything rebuilt into the buffers, then attention over them
    out_2 = torch.full_like(out_f, 9.0)
    ctx.kvd_recompute_kv_fp8(0, [(b, 0, n_old_list[b] + n_live + 1, bufs[b][0], bufs[b][1]) for b in range(batch)], kdim)
    full = [[(bufs[b][0], bufs[b][1], kdim, pos0_list[b], n_old_list[b] + n_live + 1)] for b in range(batch)]
    ctx.kvd_decode_attention(0, batch, q, q_pos, full, 0.0, out_2)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    if not keep_nothing:
        for b in range(batch):   # the stored ranges of the fused call: same bits as the plain FP8 recompute
            assert torch.equal(cur_fused[b][0], bufs[b][0][-1]) and torch.equal(cur_fused[b][1], bufs[b][1][-1])
    refs = []
    for b in range(batch):
        Kr, Vr = oracle_fp8_kv(shape, w, X_all[b], pos_all[b])
        T = X_all[b].shape[0]
        Kr, Vr = Kr.reshape(T, shape.n_kv_heads, shape.d_head), Vr.reshape(T, shape.n_kv_heads, shape.d_head)
        refs.append(oracle.decode_attention(bf16_to_f64(q_bits[b]), q_pos[b], [(Kr, Vr, int(pos_all[b][0]))],
                                            1.0 / math.sqrt(shape.d_head), shape.sliding_window))
    ctx.close()
    return host_f64(out_f), host_f64(out_2), np.stack(refs)


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, QWEN3_4B], ids=lambda s: s.name)
@pytest.mark.parametrize("n_old,n_live", [(1, 0), (100, 7), (256, 0), (257, 64), (700, 33), (1300, 256)])
def test_fused_fp8_matches_the_fp8_oracle_and_the_two_call_path(shape, n_old, n_live):
    f, two, ref = run_case(shape, [n_old], n_live, seed=n_old)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, QWEN3_4B], ids=lambda s: s.name)
def test_fused_fp8_with_nothing_kept(shape):
    # a cache budget of zero: every token, the current one included, is rebuilt from its FP8 checkpoint
    f, two, ref = run_case(shape, [600, 1, 255], 0, pos0_list=[0, 3, 77], seed=5, keep_nothing=True)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")


def test_fused_fp8_at_the_bench_size():
    f, two, ref = run_case(GEMMA3_4B_GLOBAL, [4096], 0, max_tokens=4104, seed=8)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")


def test_fused_fp8_batch_with_ragged_ranges_and_an_empty_one():
    f, two, ref = run_case(GEMMA3_4B_GLOBAL, [300, 0, 513, 40], 16, pos0_list=[0, 5, 11, 1000], seed=7)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")


def test_fused_fp8_on_a_sliding_window_layer_masks_by_stored_position():
    f, two, ref = run_case(GEMMA3_4B_LOCAL, [1500], 20, seed=9)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")


def test_fused_fp8_is_refused_without_its_store_and_for_other_shapes():
    shape = GEMMA3_4B_GLOBAL
    ctx, w = open_layer(shape, max_tokens=256, with_store=True)   # the bf16 store only
    kdim = shape.n_kv_heads * shape.d_head
    q = dev(make_query(shape, 1, seed=1))
    out = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(kvd.KvdError) as e:
        ctx.kvd_decode_attention_recompute_fp8(0, 1, q, [0], [(0, 0, 0)], [], kdim, [[]], 0.0, out)
    assert e.value.status == 5
    ctx.close()
    shape = SMOLLM2_135M  # 128-column tiles
    ctx, w = open_layer(shape, max_tokens=256)
    arena = torch.zeros(kvd.kvd_store_bytes_fp8(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena, 1)
    q = dev(make_query(shape, 1, seed=1))
    out = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(kvd.KvdError) as e:
        ctx.kvd_decode_attention_recompute_fp8(0, 1, q, [0], [(0, 0, 0)], [], shape.n_kv_heads * shape.d_head, [[]], 0.0, out)
    assert e.value.status == 6
    assert ctx.kvd_poll_status() == kvd.KVD_OK


def test_fused_fp8_decode_loop_with_nothing_kept_crosses_a_block_boundary():
    """Twelve decode steps of one sequence whose every token lives in the FP8 store only: the new row is
    quantised in, then all rows (250 -> 262, across the 256-row block boundary) are rebuilt and attended."""
    shape = GEMMA3_4B_GLOBAL
    ctx, w = open_layer(shape, max_tokens=512)
    arena = torch.zeros(kvd.kvd_store_bytes_fp8(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena, 1)
    kdim = shape.n_kv_heads * shape.d_head
    n0, steps = 250, 12
    X = make_residuals(shape, n0 + steps, seed=77, outliers=True)
    pos = np.arange(n0 + steps)
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    q_bits = make_query(shape, steps, seed=78)
    q = dev(q_bits)
    Kr, Vr = oracle_fp8_kv(shape, w, X, pos)
    Kr = Kr.reshape(-1, shape.n_kv_heads, shape.d_head)
    Vr = Vr.reshape(-1, shape.n_kv_heads, shape.d_head)
    ctx.kvd_checkpoint_residual_fp8(0, 0, x[:n0], p[:n0], n0)
    out = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    for t in range(steps):
        n = n0 + t + 1
        ctx.kvd_checkpoint_residual_fp8(0, 0, x[n - 1:n], p[n - 1:n], 1)
        assert ctx.kvd_rows_stored_fp8(0, 0) == n
        ctx.kvd_decode_attention_recompute_fp8(0, 1, q[t:t + 1], [n - 1], [(0, 0, n)], [], kdim, [[]], 0.0, out)
        ref = oracle.decode_attention(bf16_to_f64(q_bits[t]), n - 1, [(Kr[:n], Vr[:n], 0)],
                                      1.0 / math.sqrt(shape.d_head), shape.sliding_window)
        attn_check(host_f64(out)[0], ref, f"step {t}")
    assert ctx.kvd_poll_status() == kvd.KVD_OK


def test_fused_fp8_without_queries_only_stores_and_empty_call_launches_nothing():
    shape = GEMMA3_4B_GLOBAL
    ctx, w = open_layer(shape, max_tokens=512)
    arena = torch.zeros(kvd.kvd_store_bytes_fp8(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena, 1)
    kdim = shape.n_kv_heads * shape.d_head
    n = 70
    X = make_residuals(shape, n, seed=3, outliers=True)
    x, p = dev(X), torch.arange(n, dtype=torch.int32, device="cuda")
    ctx.kvd_checkpoint_residual_fp8(0, 0, x, p, n)
    before = ctx.kvd_launch_count()
    ctx.kvd_decode_attention_recompute_fp8(0, 0, None, [], [], [], kdim, [], 0.0, None)   # nothing to do
    assert ctx.kvd_launch_count() == before
    # batch 0 with ranges to store: the call is a plain FP8 recompute of those ranges
    k1 = torch.zeros((n, kdim), dtype=torch.bfloat16, device="cuda"); v1 = torch.zeros_like(k1)
    k2 = torch.zeros_like(k1); v2 = torch.zeros_like(k1)
    ctx.kvd_decode_attention_recompute_fp8(0, 0, None, [], [], [(0, 0, n, k1, v1)], kdim, [], 0.0, None)
    ctx.kvd_recompute_kv_fp8(0, [(0, 0, n, k2, v2)], kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.equal(k1, k2) and torch.equal(v1, v2) and float(k1.abs().max()) > 0


def test_fused_fp8_at_the_largest_batch_without_stored_ranges():
    # 64 sequences is the most one call takes when nothing is stored (batch + stored ranges <= 64)
    lens = [int(v) for v in np.random.default_rng(13).integers(1, 500, size=64)]
    f, two, ref = run_case(GEMMA3_4B_GLOBAL, lens, 0, pos0_list=[2 * b for b in range(64)], max_tokens=1024, seed=14,
                           keep_nothing=True)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")
    # 33 sequences with one stored range each exceed the limit of 64 ranges per call
    shape = GEMMA3_4B_GLOBAL
    ctx, w = open_layer(shape, max_tokens=64, max_batch=33, max_seqs=33)
    arena = torch.zeros(kvd.kvd_store_bytes_fp8(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena, 1)
    kdim = shape.n_kv_heads * shape.d_head
    q = dev(make_query(shape, 33, seed=1))
    out = torch.zeros((33, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((33, kdim), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(kvd.KvdError) as e:
        ctx.kvd_decode_attention_recompute_fp8(0, 33, q, [0] * 33, [(b, 0, 0) for b in range(33)],
                                               [(b, 0, 0, k[b:], k[b:]) for b in range(33)], kdim, [[] for _ in range(33)], 0.0, out)
    assert e.value.status == 4


def test_fused_fp8_with_the_new_tokens_as_caller_held_rows():
    """A batch of 5 sequences: evicted ranges attended inside the kernel, the new tokens handed over as one
    contiguous buffer of quantised rows.  Same output and same K_t, V_t bits as with the new tokens in the store."""
    shape = GEMMA3_4B_GLOBAL
    lens = [300, 0, 513, 40, 129]
    batch = len(lens)
    ctx, w = open_layer(shape, max_tokens=1024, max_batch=batch, max_seqs=batch)
    arena = torch.zeros(kvd.kvd_store_bytes_fp8(ctx.desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena, 1)
    kdim = shape.n_kv_heads * shape.d_head
    q = dev(make_query(shape, batch, seed=21))
    x_new = torch.empty((batch, shape.d_hidden), dtype=torch.bfloat16, device="cuda")
    p_new = torch.empty((batch,), dtype=torch.int32, device="cuda")
    for b, n in enumerate(lens):
        X = dev(make_residuals(shape, n + 1, seed=300 + b, outliers=True))
        p = torch.arange(n + 1, dtype=torch.int32, device="cuda") + 7 * b
        ctx.kvd_checkpoint_residual_fp8(b, 0, X, p, n + 1)      # the new token too: the reference form reads it there
        x_new[b].copy_(X[n])
        p_new[b] = n + 7 * b
    q_pos = [n + 7 * b for b, n in enumerate(lens)]
    ranges = [(b, 0, n) for b, n in enumerate(lens)]
    k_a = torch.zeros((batch, kdim), dtype=torch.bfloat16, device="cuda"); v_a = torch.zeros_like(k_a)
    k_b = torch.zeros_like(k_a); v_b = torch.zeros_like(k_a)
    out_a = torch.zeros((batch, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    out_b = torch.zeros_like(out_a)
    live = lambda k, v: [[(k[b:], v[b:], kdim, q_pos[b], 1)] for b in range(batch)]
    ctx.kvd_decode_attention_recompute_fp8(0, batch, q, q_pos, ranges, [(b, lens[b], 1, k_a[b:], v_a[b:]) for b in range(batch)],
                                           kdim, live(k_a, v_a), 0.0, out_a)
    codes = torch.zeros((batch, shape.d_hidden), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((batch,), dtype=torch.float32, device="cuda")
    sumsq = torch.zeros_like(scales)
    ctx.kvd_quantize_rows_fp8(x_new, batch, codes, scales, sumsq)
    ctx.kvd_decode_attention_recompute_fp8_rows(0, batch, q, q_pos, ranges, [], (codes, scales, sumsq, p_new, batch, k_b, v_b),
                                                kdim, live(k_b, v_b), 0.0, out_b)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.equal(k_a, k_b) and torch.equal(v_a, v_b) and torch.equal(out_a, out_b)
    assert float(out_a.abs().max()) > 0
