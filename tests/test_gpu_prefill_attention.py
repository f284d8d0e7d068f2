"""kvd_prefill_attention (many query tokens of one sequence in one launch, tiled on the tensor cores) through the C ABI.

  * every row follows the fp64 oracle called for that row alone (Eq. 6-7 with the row's own causal limit and the
    layer's window), at the attention tolerance: relative Frobenius <= 1e-2, max abs <= 1e-2 * max |oracle|;
  * a row's bits depend on the row, its position and the keys only: the same token attended alone, in a short call
    and in a long one, first or last of its tile, gives identical bits;
  * segments, gaps between segments, rows beyond the last key, rows without a visible key (zeros), group sizes 1-8.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from kvd_synth import (LayerShape, GEMMA3_4B_GLOBAL, GEMMA3_4B_LOCAL, QWEN3_4B, SMOLLM2_135M, TINY_GQA, TINY_MHA, bf16_to_f64,
                       make_kv, make_query)
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
