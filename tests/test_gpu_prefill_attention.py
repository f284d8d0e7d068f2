"""kvd_prefill_attention (many query tokens of one sequence in one launch, tiled on the tensor cores) through the C ABI.

  * every row follows the fp64 oracle called for that row alone (Eq. 6-7 with the row's own causal limit and the
    layer's window), at the attention tolerance: relative Frobenius <= 1e-2, max abs <= 1e-2 * max |oracle|;
  * a row's bits depend on the row, its position and the keys only: the same token attended alone, in a short call
    and in a long one, first or last of its tile, gives identical bits;
  * segments, gaps between segments, rows beyond the last key, rows without a visible key (zeros), group sizes 1-8;
  * keys whose magnitude grows or shrinks from block to block (the lazily followed maximum and the rescale of the
    accumulated output), odd tile counts, calls far longer than the sliding window, shuffled query rows, fp16.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from kvd_synth import (LayerShape, GEMMA3_4B_GLOBAL, GEMMA3_4B_LOCAL, QWEN3_4B, SMOLLM2_135M, TINY_GQA, TINY_MHA, bf16_to_f64,
                       f32_to_bf16_bits, make_kv, make_layer_weights, make_query)
from gpu_util import dev, host_f64, open_layer

pytestmark = pytest.mark.gpu


def attn_check(got, ref):
    d = got - ref
    assert np.linalg.norm(d) <= 1e-2 * np.linalg.norm(ref), np.linalg.norm(d) / np.linalg.norm(ref)
    assert np.max(np.abs(d)) <= 1e-2 * np.max(np.abs(ref)) + 1e-30


def oracle_rows(shape, q_bits, q_pos, seg_bits, rows):
    outs = []
    segs = [(bf16_to_f64(K), bf16_to_f64(V), first) for (K, V, first) in seg_bits if K.shape[0] > 0]
    for i in rows:
        outs.append(oracle.decode_attention(bf16_to_f64(q_bits[i]), int(q_pos[i]), segs, 1.0 / math.sqrt(shape.d_head),
                                            shape.sliding_window))
    return np.stack(outs)


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, GEMMA3_4B_LOCAL, QWEN3_4B, SMOLLM2_135M, TINY_GQA, TINY_MHA], ids=lambda s: s.name)
def test_rows_follow_the_oracle_and_do_not_depend_on_each_other(shape):
    T = 1300 if shape.d_head > 64 else 700
    ctx, _ = open_layer(shape, max_tokens=4096)
    kdim = shape.n_kv_heads * shape.d_head
    K, V = make_kv(shape, T, seed=15)
    cut1, cut2 = 300, 310  # positions 300..309 are held by no segment (a gap)
    seg_bits = [(K[:cut1], V[:cut1], 0), (K[cut2:T - 1], V[cut2:T - 1], cut2), (K[T - 1:], V[T - 1:], T - 1)]
    kd = [(dev(k), dev(v)) for k, v, _ in seg_bits]
    segs = [(kd[i][0], kd[i][1], kdim, seg_bits[i][2], seg_bits[i][0].shape[0]) for i in range(3)]
    rng = np.random.default_rng(21)
    q_pos = np.sort(np.concatenate([[0, 1, 63, 64, 299, 305, 310, T - 1, T + 50], rng.choice(np.arange(2, T), 120, replace=False)]))
    n = len(q_pos)
    q_bits = make_query(shape, n, seed=16)
    q, qp = dev(q_bits), torch.from_numpy(q_pos.astype(np.int32)).cuda()
    out = torch.full((n, shape.n_q_heads, shape.d_head), 9.0, dtype=torch.bfloat16, device="cuda")
    n0 = ctx.kvd_launch_count()
    ctx.kvd_prefill_attention(0, n, q, qp, segs, 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK and ctx.kvd_launch_count() - n0 == 1
    sample = sorted(set([0, 1, 2, 3, 4, 5, 6, 7, n - 2, n - 1] + rng.choice(n, 14, replace=False).tolist()))
    attn_check(host_f64(out[torch.tensor(sample).cuda()]), oracle_rows(shape, q_bits, q_pos, seg_bits, sample))
    # the same rows alone, and as a short call starting somewhere else in a tile
    one = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    for i in (0, 5, 17, 64, n - 1):
        ctx.kvd_prefill_attention(0, 1, q[i:i + 1], qp[i:i + 1], segs, 0.0, one)
        assert torch.equal(one[0], out[i]), i
    few = torch.zeros((7, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_prefill_attention(0, 7, q[30:37], qp[30:37], segs, 0.0, few)
    assert torch.equal(few, out[30:37])
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    ctx.close()


def test_causal_prefill_of_consecutive_tokens_and_rows_without_keys():
    shape = GEMMA3_4B_GLOBAL
    ctx, _ = open_layer(shape, max_tokens=2048)
    kdim = shape.n_kv_heads * shape.d_head
    T = 600
    K, V = make_kv(shape, T, seed=3)
    k, v = dev(K), dev(V)
    # a segment of 600 tokens attending causally to itself, keys starting at position 40
    q_pos = np.arange(T) + 40
    q_pos[:3] = [0, 10, 39]  # three tokens before the first key: nothing visible -> zeros
    q_bits = make_query(shape, T, seed=4)
    out = torch.full((T, shape.n_q_heads, shape.d_head), 9.0, dtype=torch.bfloat16, device="cuda")
    ctx.kvd_prefill_attention(0, T, dev(q_bits), torch.from_numpy(q_pos.astype(np.int32)).cuda(), [(k, v, kdim, 40, T)], 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.all(out[:3] == 0)
    sample = [3, 4, 66, 67, 300, T - 1]
    attn_check(host_f64(out[torch.tensor(sample).cuda()]), oracle_rows(shape, q_bits, q_pos, [(K, V, 40)], sample))
    ctx.close()


@pytest.mark.parametrize("group", [1, 2, 3, 4, 8])
def test_group_sizes(group):
    shape = LayerShape(f"g{group}", 128, 2 * group, 2, 64, 1e-6, False, 1.0e4)
    ctx, _ = open_layer(shape, max_tokens=512)
    kdim = shape.n_kv_heads * shape.d_head
    T = 200
    K, V = make_kv(shape, T, seed=group)
    q_pos = np.arange(T)
    q_bits = make_query(shape, T, seed=group + 10)
    out = torch.zeros((T, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_prefill_attention(0, T, dev(q_bits), torch.from_numpy(q_pos.astype(np.int32)).cuda(), [(dev(K), dev(V), kdim, 0, T)], 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    sample = [0, 1, 15, 16, 63, 64, 65, 199]
    attn_check(host_f64(out[torch.tensor(sample).cuda()]), oracle_rows(shape, q_bits, q_pos, [(K, V, 0)], sample))
    ctx.close()


@pytest.mark.parametrize("ramp", ["up", "down"])
def test_scores_whose_maximum_jumps_by_large_factors(ramp):
    """The kernel follows a row's maximum lazily (its reference moves only when a block exceeds it by 2^8) and
    rescales what it has accumulated when it does: keys whose magnitude grows from block to block force that path in
    every block, keys that shrink never take it again after the first; both must follow Eq. 6-7."""
    shape = QWEN3_4B
    ctx, _ = open_layer(shape, max_tokens=2048)
    kdim = shape.n_kv_heads * shape.d_head
    T = 700
    K, V = make_kv(shape, T, seed=31)
    kf = bf16_to_f64(K)
    growth = 1.6 ** (np.arange(T) // 64)                       # x 1.6 per 64-key block: 11 blocks span a factor of 110
    kf = kf * (growth if ramp == "up" else growth[::-1])[:, None, None]
    K = f32_to_bf16_bits(kf.astype(np.float32))
    q_pos = np.arange(T)
    q_bits = make_query(shape, T, seed=32)
    out = torch.zeros((T, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_prefill_attention(0, T, dev(q_bits), torch.from_numpy(q_pos.astype(np.int32)).cuda(), [(dev(K), dev(V), kdim, 0, T)], 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    sample = [0, 63, 64, 130, 257, 448, 449, 640, T - 1]
    attn_check(host_f64(out[torch.tensor(sample).cuda()]), oracle_rows(shape, q_bits, q_pos, [(K, V, 0)], sample))
    ctx.close()


@pytest.mark.parametrize("shape,T", [(GEMMA3_4B_GLOBAL, 64 * 5 + 7), (GEMMA3_4B_LOCAL, 2500), (QWEN3_4B, 32 * 7), (SMOLLM2_135M, 32 * 3 + 1)],
                         ids=lambda v: getattr(v, "name", str(v)))
def test_odd_numbers_of_tiles_long_rows_and_unsorted_positions(shape, T):
    """Tile counts that are odd, a call much longer than the sliding window (tiles that start far from position 0),
    and query rows given in a shuffled order: every sampled row follows the oracle, and the shuffled call returns the
    bits of the ordered one row for row."""
    ctx, _ = open_layer(shape, max_tokens=4096)
    kdim = shape.n_kv_heads * shape.d_head
    K, V = make_kv(shape, T, seed=41)
    k, v = dev(K), dev(V)
    q_bits = make_query(shape, T, seed=42)
    q_pos = np.arange(T)
    out = torch.zeros((T, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_prefill_attention(0, T, dev(q_bits), torch.from_numpy(q_pos.astype(np.int32)).cuda(), [(k, v, kdim, 0, T)], 0.0, out)
    rng = np.random.default_rng(43)
    sample = sorted(set([0, 1, T // 2, T - 2, T - 1] + rng.choice(T, 10, replace=False).tolist()))
    attn_check(host_f64(out[torch.tensor(sample).cuda()]), oracle_rows(shape, q_bits, q_pos, [(K, V, 0)], sample))
    perm = rng.permutation(T)
    out2 = torch.zeros_like(out)
    ctx.kvd_prefill_attention(0, T, dev(q_bits[perm]), torch.from_numpy(q_pos[perm].astype(np.int32)).cuda(), [(k, v, kdim, 0, T)], 0.0, out2)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.equal(out2, out[torch.from_numpy(perm).cuda()])
    ctx.close()


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, QWEN3_4B, SMOLLM2_135M], ids=lambda s: s.name)
def test_fp16_prefill_attention_follows_the_oracle(shape):
    w = make_layer_weights(shape)
    desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                         shape.qk_norm, shape.rms_eps, shape.rope_style, 1, 2048, 1)
    ctx = kvd.Kvd(desc)
    ctx.kvd_set_dtype(1)
    to16 = lambda bits: torch.from_numpy(bf16_to_f64(bits).astype(np.float16)).cuda()
    ctx.kvd_set_layer(0, to16(w.w_kv), to16(w.gamma_in), to16(w.gamma_k) if w.gamma_k is not None else None, shape.rope_theta,
                      shape.sliding_window)
    kdim = shape.n_kv_heads * shape.d_head
    T = 333
    rng = np.random.default_rng(7)
    q16 = rng.standard_normal((T, shape.n_q_heads, shape.d_head)).astype(np.float16)
    k16 = rng.standard_normal((T, kdim)).astype(np.float16)
    v16 = rng.standard_normal((T, kdim)).astype(np.float16)
    q_pos = np.arange(T) + 9
    out = torch.zeros((T, shape.n_q_heads, shape.d_head), dtype=torch.float16, device="cuda")
    ctx.kvd_prefill_attention(0, T, torch.from_numpy(q16).cuda(), torch.from_numpy(q_pos.astype(np.int32)).cuda(),
                              [(torch.from_numpy(k16).cuda(), torch.from_numpy(v16).cuda(), kdim, 9, T)], 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    sample = [0, 1, 63, 64, 65, 200, T - 1]
    kv = (k16.astype(np.float64).reshape(T, shape.n_kv_heads, shape.d_head), v16.astype(np.float64).reshape(T, shape.n_kv_heads, shape.d_head), 9)
    ref = np.stack([oracle.decode_attention(q16[i].astype(np.float64), int(q_pos[i]), [kv], 1.0 / math.sqrt(shape.d_head),
                                            shape.sliding_window) for i in sample])
    attn_check(out[torch.tensor(sample).cuda()].double().cpu().numpy(), ref)
    ctx.close()


def test_full_size_call_of_the_benchmark_on_sampled_rows():
    """The launch `bench.py` times (key prefill_attention): 16384 tokens of the Gemma-shaped global layer attending to
    themselves, 256 tiles in 128 CTA pairs per KV head.  Rows sampled across the call -- first and last rows of tiles,
    of pairs, of the call -- against the fp64 oracle called for each row alone."""
    shape = GEMMA3_4B_GLOBAL
    T = 16384
    ctx, _ = open_layer(shape, max_tokens=T + 8)
    kdim = shape.n_kv_heads * shape.d_head
    K, V = make_kv(shape, T, seed=61)
    q_bits = make_query(shape, T, seed=62)
    q_pos = np.arange(T)
    out = torch.zeros((T, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_prefill_attention(0, T, dev(q_bits), torch.from_numpy(q_pos.astype(np.int32)).cuda(), [(dev(K), dev(V), kdim, 0, T)], 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    rng = np.random.default_rng(63)
    sample = sorted(set([0, 63, 64, 127, 128, 8191, 8192, T - 129, T - 128, T - 65, T - 64, T - 1] + rng.choice(T, 12, replace=False).tolist()))
    attn_check(host_f64(out[torch.tensor(sample).cuda()]), oracle_rows(shape, q_bits, q_pos, [(K, V, 0)], sample))
    ctx.close()


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, QWEN3_4B, SMOLLM2_135M], ids=lambda s: s.name)
def test_no_keys_at_all_gives_zeros_and_an_empty_call_is_accepted(shape):
    ctx, _ = open_layer(shape, max_tokens=256)
    kdim = shape.n_kv_heads * shape.d_head
    n = 70
    q = dev(make_query(shape, n, seed=5))
    qp = torch.arange(n, dtype=torch.int32, device="cuda")
    out = torch.full((n, shape.n_q_heads, shape.d_head), 3.0, dtype=torch.bfloat16, device="cuda")
    ctx.kvd_prefill_attention(0, n, q, qp, [], 0.0, out)                       # no segment
    assert torch.all(out == 0)
    K, V = make_kv(shape, 8, seed=6)
    out.fill_(3.0)
    ctx.kvd_prefill_attention(0, n, q, qp, [(dev(K), dev(V), kdim, 100, 0)], 0.0, out)   # a segment of length zero
    assert torch.all(out == 0)
    out.fill_(3.0)
    ctx.kvd_prefill_attention(0, n, q, qp, [(dev(K), dev(V), kdim, 100, 8)], 0.0, out)   # every key lies after every row
    assert torch.all(out == 0)
    ctx.kvd_prefill_attention(0, 0, q, qp, [], 0.0, out)                       # nothing to do
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    ctx.close()


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, QWEN3_4B], ids=lambda s: s.name)
def test_repeated_launches_give_the_same_bits(shape):
    """Nothing in the kernel depends on timing: which softmax group is ahead, when a block lands, in which order the
    CTAs start.  Thirty launches of a 3000-token call (pairs and single CTAs, several waves) return identical bits."""
    T = 3000
    ctx, _ = open_layer(shape, max_tokens=T + 8)
    kdim = shape.n_kv_heads * shape.d_head
    K, V = make_kv(shape, T, seed=71)
    k, v = dev(K), dev(V)
    q = dev(make_query(shape, T, seed=72))
    qp = torch.arange(T, dtype=torch.int32, device="cuda")
    first = torch.zeros((T, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_prefill_attention(0, T, q, qp, [(k, v, kdim, 0, T)], 0.0, first)
    out = torch.zeros_like(first)
    for _ in range(30):
        out.fill_(1.0)
        ctx.kvd_prefill_attention(0, T, q, qp, [(k, v, kdim, 0, T)], 0.0, out)
        assert torch.equal(out, first)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    ctx.close()
