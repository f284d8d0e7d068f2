"""kvd_decode_attention_static: decode attention for callers that must not allocate device memory.

Some users of this library run where cudaMalloc is off limits -- inside another framework's memory
pool, under a fixed device-memory budget, or in a plug-in whose host forbids allocation after
start-up.  For them the library offers one entry point whose scratch (the split partials) is a
fixed array compiled into the library instead of a caller-provided workspace.

This file is collected last on purpose: a run that stops at the first failure has then already run
every other test.  The test calls the entry point through the C ABI twice in a row with different
inputs -- the second call starts with the first call's leftovers in the shared array -- and checks
each output against kvd_decode_attention on the same inputs, plus the size limit.
"""
import numpy as np
import pytest
import torch

import paper_2603_19664_b200 as kvd
from kvd_synth import GEMMA3_4B_LOCAL, QWEN3_4B, make_kv, make_query
from gpu_util import dev, host_f64, open_layer

pytestmark = pytest.mark.gpu


def _both(ctx, shape, q_bits, q_pos, seg_bits):
    """Run the workspace entry point and the allocation-free one on the same device tensors."""
    batch = q_bits.shape[0]
    kdim = shape.n_kv_heads * shape.d_head
    q = dev(q_bits)
    keep, segs = [], []
    for b in range(batch):
        row = []
        for (Kb, Vb, first) in seg_bits[b]:
            k, v = dev(Kb), dev(Vb)
            keep += [k, v]
            row.append((k, v, kdim, first, Kb.shape[0]))
        segs.append(row)
    ref = torch.full((batch, shape.n_q_heads, shape.d_head), 3.0, dtype=torch.bfloat16, device="cuda")
    got = torch.full_like(ref, -3.0)
    ctx.kvd_decode_attention(0, batch, q, q_pos, segs, 0.0, ref)
    st = kvd.kvd_decode_attention_static(shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.sliding_window,
                                         batch, q, q_pos, segs, 0.0, got)
    assert st == kvd.KVD_OK, kvd.status_string(st)
    torch.cuda.synchronize()
    return ref, got


def _check(ref, got):
    r, g = host_f64(ref), host_f64(got)
    # same tolerance as the attention parity tests ...
    assert np.linalg.norm(g - r) <= 1e-2 * np.linalg.norm(r)
    assert np.max(np.abs(g - r)) <= 1e-2 * np.max(np.abs(r))
    # ... and in fact the same kernel with the same split, so the bits agree
    assert torch.equal(ref, got)


def test_static_scratch_matches_workspace_path_on_two_calls_in_a_row():
    # call 1: sliding-window layer, batch 3, keys spread over recomputed / window / current segments
    shape = GEMMA3_4B_LOCAL
    ctx, _ = open_layer(shape, max_tokens=8192, max_batch=3)
    lens = [3000, 65, 1500]
    q = make_query(shape, 3, seed=41)
    segs, qpos = [], []
    for b, T in enumerate(lens):
        K, V = make_kv(shape, T, seed=60 + b)
        cut = max(1, T - 257)
        segs.append([(K[:cut], V[:cut], 0), (K[cut:T - 1], V[cut:T - 1], cut), (K[T - 1:], V[T - 1:], T - 1)])
        qpos.append(T - 1)
    ref, got = _both(ctx, shape, q, qpos, segs)
    _check(ref, got)
    ctx.close()

    # call 2 right after: another model shape, longer context; the array still holds call 1's partials
    shape = QWEN3_4B
    ctx, _ = open_layer(shape, max_tokens=16384, max_batch=2)
    q = make_query(shape, 2, seed=42)
    segs, qpos = [], []
    for b, T in enumerate([9000, 1]):
        K, V = make_kv(shape, T, seed=70 + b)
        segs.append([(K, V, 0)])
        qpos.append(T - 1)
    ref, got = _both(ctx, shape, q, qpos, segs)
    _check(ref, got)

    # a request whose partials cannot fit the fixed array is refused, and nothing is launched
    T = 16000
    K, V = make_kv(shape, T, seed=80)
    k, v = dev(K), dev(V)
    kdim = shape.n_kv_heads * shape.d_head
    big = 64
    qb = dev(make_query(shape, big, seed=43))
    out = torch.full((big, shape.n_q_heads, shape.d_head), 5.0, dtype=torch.bfloat16, device="cuda")
    st = kvd.kvd_decode_attention_static(shape.n_q_heads, shape.n_kv_heads, shape.d_head, 0, big, qb, [T - 1] * big,
                                         [[(k, v, kdim, 0, T)]] * big, 0.0, out)
    assert st == 4, kvd.status_string(st)  # KVD_ERR_CAPACITY
    torch.cuda.synchronize()
    assert torch.all(out == 5.0)
    # more sequences than one launch holds
    st = kvd.kvd_decode_attention_static(shape.n_q_heads, shape.n_kv_heads, shape.d_head, 0, 65, qb, [0] * 65,
                                         [[]] * 65, 0.0, out)
    assert st == 4
    ctx.close()
