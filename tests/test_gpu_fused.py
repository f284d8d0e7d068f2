"""GPU parity of kvd_decode_attention_recompute (recompute fused into attention) through the C ABI.

The call must give attention over [K/V recomputed from store ranges] + [live segments]:
  * against the fp64 oracle (oracle.recompute_kv for every key, then oracle.decode_attention), with the
    attention tolerance: rel Frobenius <= 1e-2 and max abs <= 1e-2 * max |oracle|;
  * against the two-call GPU path (kvd_recompute_kv_step + kvd_decode_attention), to which it is
    equal up to rounding (the fused kernel splits the recomputed keys by 256-row blocks and does not
    round K/V to bf16 in between), with the same tolerance.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from kvd_synth import GEMMA3_4B_GLOBAL, GEMMA3_4B_LOCAL, QWEN3_4B, SMOLLM2_135M, bf16_to_f64, make_query, make_residuals
from gpu_util import dev, host_f64, open_layer, oracle_kv

pytestmark = pytest.mark.gpu


def attn_check(got, ref, what=""):
    d = got - ref
    rel = np.linalg.norm(d) / max(np.linalg.norm(ref), 1e-300)
    assert rel <= 1e-2, f"{what} rel {rel}"
    assert np.max(np.abs(d)) <= 1e-2 * np.max(np.abs(ref)) + 1e-30, f"{what} max abs {np.max(np.abs(d))}"


def run_case(shape, n_old_list, n_live, pos0_list=None, max_tokens=4096, seed=1):
    """One decode step of a batch: sequence b has n_old_list[b] evicted rows in the store (positions
    pos0 .. pos0+n_old-1), n_live live keys after them (recomputed into a K/V buffer beforehand) and the
    current token.  Returns (fused out, two-call out, oracle out)."""
    batch = len(n_old_list)
    ctx, w = open_layer(shape, max_tokens=max_tokens, max_batch=batch, max_seqs=batch, with_store=True)
    kdim = shape.n_kv_heads * shape.d_head
    pos0_list = pos0_list or [0] * batch
    q_bits = make_query(shape, batch, seed=seed)
    q = dev(q_bits)
    X_all, pos_all, keep = [], [], []
    x_cur = torch.empty((batch, shape.d_hidden), dtype=torch.bfloat16, device="cuda")
    p_cur = torch.empty((batch,), dtype=torch.int32, device="cuda")
    k_cur = torch.zeros((batch, kdim), dtype=torch.bfloat16, device="cuda")
    v_cur = torch.zeros_like(k_cur)
    q_pos, live, ranges_fused, ranges_plain, old_bufs = [], [], [], [], []
    for b in range(batch):
        n_old, T = n_old_list[b], n_old_list[b] + n_live + 1
        X = make_residuals(shape, T, seed=seed * 100 + b, outliers=True)
        pos = np.arange(T) + pos0_list[b]
        X_all.append(X)
        pos_all.append(pos)
        x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
        keep += [x, p]
        if n_old:
            ctx.kvd_checkpoint_residual(b, 0, x[:n_old], p[:n_old], n_old)
        # live keys: K/V computed beforehand (they are the cache window)
        kl = torch.zeros((max(n_live, 1), kdim), dtype=torch.bfloat16, device="cuda")
        vl = torch.zeros_like(kl)
        if n_live:
            ctx.kvd_recompute_kv(0, x[n_old:n_old + n_live], p[n_old:n_old + n_live], n_live, kl, vl, kdim)
        x_cur[b].copy_(x[T - 1])
        p_cur[b] = int(pos[T - 1])
        q_pos.append(int(pos[T - 1]))
        live.append((kl, vl))
        ko = torch.zeros((max(n_old, 1), kdim), dtype=torch.bfloat16, device="cuda")
        vo = torch.zeros_like(ko)
        old_bufs.append((ko, vo))
        ranges_fused.append((b, 0, n_old))
        ranges_plain.append((b, 0, n_old, ko, vo))

    def segs(with_old):
        out = []
        for b in range(batch):
            n_old = n_old_list[b]
            row = []
            if with_old and n_old:
                row.append((old_bufs[b][0], old_bufs[b][1], kdim, pos0_list[b], n_old))
            if n_live:
                row.append((live[b][0], live[b][1], kdim, pos0_list[b] + n_old, n_live))
            row.append((k_cur[b:b + 1], v_cur[b:b + 1], kdim, q_pos[b], 1))
            out.append(row)
        return out

    out_f = torch.full((batch, shape.n_q_heads, shape.d_head), 9.0, dtype=torch.bfloat16, device="cuda")
    ctx.kvd_decode_attention_recompute(0, batch, q, q_pos, ranges_fused, x_cur, p_cur, batch, k_cur, v_cur, kdim,
                                       segs(False), 0.0, out_f)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    k_cur_fused = k_cur.clone()
    # the two-call path on the same inputs
    out_2 = torch.full_like(out_f, 9.0)
    ctx.kvd_recompute_kv_step(0, [r for r in ranges_plain if r[2] > 0], x_cur, p_cur, batch, k_cur, v_cur, kdim)
    ctx.kvd_decode_attention(0, batch, q, q_pos, segs(True), 0.0, out_2)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.equal(k_cur, k_cur_fused)  # the new tokens' K are written by the fused call, same bits
    # oracle
    refs = []
    for b in range(batch):
        Kr, Vr = oracle_kv(shape, w, X_all[b], pos_all[b])
        T = X_all[b].shape[0]
        Kr, Vr = Kr.reshape(T, shape.n_kv_heads, shape.d_head), Vr.reshape(T, shape.n_kv_heads, shape.d_head)
        refs.append(oracle.decode_attention(bf16_to_f64(q_bits[b]), q_pos[b], [(Kr, Vr, int(pos_all[b][0]))],
                                            1.0 / math.sqrt(shape.d_head), shape.sliding_window))
    ctx.close()
    return host_f64(out_f), host_f64(out_2), np.stack(refs)


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, QWEN3_4B], ids=lambda s: s.name)
@pytest.mark.parametrize("n_old,n_live", [(1, 0), (100, 7), (256, 0), (257, 64), (700, 33), (1300, 256)])
def test_fused_matches_the_oracle_and_the_two_call_path(shape, n_old, n_live):
    f, two, ref = run_case(shape, [n_old], n_live, seed=n_old)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")


def test_fused_at_the_bench_size():
    # the configuration bench.py times: 4096 evicted rows + the current token, Gemma-3-4B-shaped global layer
    f, two, ref = run_case(GEMMA3_4B_GLOBAL, [4096], 0, max_tokens=4104, seed=8)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")


def test_fused_batch_with_ragged_ranges_and_an_empty_one():
    f, two, ref = run_case(GEMMA3_4B_GLOBAL, [300, 0, 513, 40], 16, pos0_list=[0, 5, 11, 1000], seed=7)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")


def test_fused_on_a_sliding_window_layer_masks_by_stored_position():
    # window 1024 on the local layer: of 1500 evicted + 20 live + 1 current keys only the last 1024 are visible
    f, two, ref = run_case(GEMMA3_4B_LOCAL, [1500], 20, seed=9)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")


def test_fused_is_refused_for_shapes_it_is_not_built_for():
    shape = SMOLLM2_135M  # 128-column tiles
    ctx, w = open_layer(shape, max_tokens=256, with_store=True)
    kdim = shape.n_kv_heads * shape.d_head
    q = dev(make_query(shape, 1, seed=1))
    out = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(kvd.KvdError) as e:
        ctx.kvd_decode_attention_recompute(0, 1, q, [0], [(0, 0, 0)], None, None, 0, None, None, kdim, [[]], 0.0, out)
    assert e.value.status == 6
    assert ctx.kvd_poll_status() == kvd.KVD_OK


def test_fused_at_the_largest_batch():
    # 64 sequences (the most one call takes), lengths 0 ... 600 evicted rows, 8 live keys each
    lens = [int(v) for v in np.random.default_rng(11).integers(0, 601, size=64)]
    lens[5], lens[40] = 0, 600
    f, two, ref = run_case(GEMMA3_4B_GLOBAL, lens, 8, pos0_list=[3 * b for b in range(64)], max_tokens=1024, seed=12)
    attn_check(f, ref, "fused vs oracle")
    attn_check(f, two, "fused vs two-call")


@pytest.mark.parametrize("shape,T", [(GEMMA3_4B_GLOBAL, 700), (QWEN3_4B, 1300)], ids=lambda x: getattr(x, "name", x))
def test_fused_with_the_current_token_inside_the_range_needs_no_live_segment(shape, T):
    """Budget zero, the form the benchmark times: every token's row is checkpointed, the current one included,
    and ranges[b] covers all T + 1 of them; the caller's row still yields K_t, V_t (same bits as
    kvd_recompute_kv), no segment is passed, and only two kernels run (recompute+attend, merge)."""
    ctx, w = open_layer(shape, max_tokens=2048, with_store=True)
    kdim = shape.n_kv_heads * shape.d_head
    X = make_residuals(shape, T + 1, seed=77, outliers=True)
    pos = np.arange(T + 1)
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    ctx.kvd_checkpoint_residual(0, 0, x, p, T + 1)
    q_bits = make_query(shape, 1, seed=77)
    q = dev(q_bits)
    out = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    kc = torch.zeros((1, kdim), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    n0 = ctx.kvd_launch_count()
    ctx.kvd_decode_attention_recompute(0, 1, q, [T], [(0, 0, T + 1)], x[T:], p[T:], 1, kc, vc, kdim, [[]], 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert ctx.kvd_launch_count() - n0 == 2
    Kr, Vr = oracle_kv(shape, w, X, pos)
    ref = oracle.decode_attention(bf16_to_f64(q_bits[0]), T, [(Kr, Vr, 0)], 1.0 / math.sqrt(shape.d_head), shape.sliding_window)
    attn_check(host_f64(out)[0], ref, "folded")
    k2 = torch.zeros_like(kc)
    v2 = torch.zeros_like(vc)
    ctx.kvd_recompute_kv(0, x[T:], p[T:], 1, k2, v2, kdim)
    assert torch.equal(kc, k2) and torch.equal(vc, v2)
    ctx.close()
