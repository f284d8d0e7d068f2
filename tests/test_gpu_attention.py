"""GPU parity of kvd_decode_attention against the fp64 oracle (through the C ABI).

Tolerance (bf16 output against the fp64 oracle on the same bf16 inputs):
    ||gpu - oracle||_F / ||oracle||_F <= 1e-2   and   max |gpu - oracle| <= 1e-2 * max |oracle|.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from kvd_synth import (LayerShape, GEMMA3_4B_GLOBAL, GEMMA3_4B_LOCAL, QWEN3_4B, SMOLLM2_135M, TINY_GQA, TINY_MHA, bf16_to_f64,
                       make_kv, make_query, make_residuals)
from gpu_util import dev, host_bits, host_f64, open_layer, oracle_kv

pytestmark = pytest.mark.gpu


def attn_check(got, ref):
    d = got - ref
    rel = np.linalg.norm(d) / max(np.linalg.norm(ref), 1e-300)
    assert rel <= 1e-2, f"rel {rel}"
    assert np.max(np.abs(d)) <= 1e-2 * np.max(np.abs(ref)) + 1e-30, f"max abs {np.max(np.abs(d))}"


def gpu_attention(ctx, shape, q_bits, q_pos, seg_lists, scale=0.0):
    """seg_lists[b] = list of (K_bits, V_bits, first_pos); returns (bf16 out tensor, kept tensors)."""
    batch = q_bits.shape[0]
    kdim = shape.n_kv_heads * shape.d_head
    q = dev(q_bits)
    out = torch.full((batch, shape.n_q_heads, shape.d_head), 9.0, dtype=torch.bfloat16, device="cuda")
    keep, segs = [], []
    for b in range(batch):
        row = []
        for (Kb, Vb, first) in seg_lists[b]:
            k, v = dev(Kb), dev(Vb)
            keep += [k, v]
            row.append((k, v, kdim, first, Kb.shape[0]))
        segs.append(row)
    ctx.kvd_decode_attention(0, batch, q, q_pos, segs, scale, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    return out


def oracle_attention(shape, q_bits, q_pos, seg_lists, window=None):
    outs = []
    for b in range(q_bits.shape[0]):
        segs = [(bf16_to_f64(K), bf16_to_f64(V), first) for (K, V, first) in seg_lists[b] if K.shape[0] > 0]
        outs.append(oracle.decode_attention(bf16_to_f64(q_bits[b]), int(q_pos[b]), segs,
                                            1.0 / math.sqrt(shape.d_head),
                                            shape.sliding_window if window is None else window))
    return np.stack(outs)


@pytest.mark.parametrize("shape", [TINY_GQA, TINY_MHA, SMOLLM2_135M, QWEN3_4B, GEMMA3_4B_GLOBAL], ids=lambda s: s.name)
@pytest.mark.parametrize("T", [1, 2, 63, 64, 65, 257, 1000])
def test_lengths_across_chunk_boundaries(shape, T):
    ctx, _ = open_layer(shape, max_tokens=4096)
    K, V = make_kv(shape, T, seed=T)
    q = make_query(shape, 1, seed=T)
    segs = [[(K, V, 0)]]
    out = gpu_attention(ctx, shape, q, [T - 1], segs)
    attn_check(host_f64(out), oracle_attention(shape, q, [T - 1], segs))


def test_config1_recompute_then_attend():
    # SmolLM2 layer: K/V of 512 tokens recomputed on the GPU, one current token, query at position 512
    shape = SMOLLM2_135M
    ctx, w = open_layer(shape, max_tokens=1024)
    kdim = shape.n_kv_heads * shape.d_head
    X = make_residuals(shape, 513, seed=1)
    pos = np.arange(513)
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    k = torch.empty((513, kdim), dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(k)
    ctx.kvd_recompute_kv(0, x[:512], p[:512], 512, k[:512], v[:512], kdim)       # RECOMPUTE_KV
    ctx.kvd_recompute_kv(0, x[512:], p[512:], 1, k[512:], v[512:], kdim)         # K_t, V_t
    q = make_query(shape, 1, seed=1)
    out = torch.empty((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_decode_attention(0, 1, dev(q), [512], [[(k[:512], v[:512], kdim, 0, 512), (k[512:], v[512:], kdim, 512, 1)]],
                             0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    # oracle chain: fp64 K/V from the residual rows, then fp64 attention
    Kr, Vr = oracle_kv(shape, w, X, pos)
    ref = oracle.decode_attention(bf16_to_f64(q[0]), 512, [(Kr[:512], Vr[:512], 0), (Kr[512:], Vr[512:], 512)],
                                  1.0 / math.sqrt(shape.d_head))
    attn_check(host_f64(out)[0], ref)


@pytest.mark.parametrize("shape,T", [(GEMMA3_4B_GLOBAL, 4096), (GEMMA3_4B_LOCAL, 4096), (GEMMA3_4B_GLOBAL, 32768),
                                     (QWEN3_4B, 8200)], ids=lambda x: getattr(x, "name", x))
def test_config2_full_size_keys(shape, T):
    ctx, _ = open_layer(shape, max_tokens=32768 + 8)
    K, V = make_kv(shape, T + 1, seed=9)
    q = make_query(shape, 1, seed=9)
    segs = [[(K[:T], V[:T], 0), (K[T:], V[T:], T)]]
    out = gpu_attention(ctx, shape, q, [T], segs)
    attn_check(host_f64(out), oracle_attention(shape, q, [T], segs))


def test_batch_with_mixed_lengths_windows_and_gaps():
    shape = GEMMA3_4B_LOCAL  # window 1024
    ctx, _ = open_layer(shape, max_tokens=8192, max_batch=5)
    lens = [1500, 70, 1024, 3000, 1]
    q = make_query(shape, 5, seed=3)
    segs, qpos = [], []
    for b, T in enumerate(lens):
        K, V = make_kv(shape, T, seed=20 + b)
        if b == 3:
            # recomputed prefix, live window, current token -- with keys after q_pos that must be ignored
            segs.append([(K[:2000], V[:2000], 0), (K[2000:2999], V[2000:2999], 2000), (K[2999:], V[2999:], 2999)])
            qpos.append(2990)
        elif b == 0:
            # a hole in the positions: 0..699 and 800..1599
            segs.append([(K[:700], V[:700], 0), (K[700:], V[700:], 800)])
            qpos.append(1599)
        else:
            segs.append([(K, V, 0)])
            qpos.append(T - 1)
    out = gpu_attention(ctx, shape, q, qpos, segs)
    ref = oracle_attention(shape, q, qpos, segs)
    for b in range(5):
        attn_check(host_f64(out)[b], ref[b])


# every supported group size on both streaming kernels (fp32 pipes; tensor cores for 3+ query heads per
# KV head at d_head <= 128), including the widest group and a sliding window
WIDE_SHAPES = [LayerShape("g8-d128", 256, 16, 2, 128, 1e-6, False, 1.0e4),
               LayerShape("g8-d64", 256, 8, 1, 64, 1e-6, False, 1.0e4, 300),
               LayerShape("g3-d128", 256, 6, 2, 128, 1e-6, False, 1.0e4),
               LayerShape("g4-d256", 256, 8, 2, 256, 1e-6, False, 1.0e4),
               LayerShape("g8-d256", 256, 8, 1, 256, 1e-6, False, 1.0e4),
               LayerShape("g1-d128", 256, 2, 2, 128, 1e-6, False, 1.0e4)]


@pytest.mark.parametrize("shape", WIDE_SHAPES, ids=lambda s: s.name)
def test_group_sizes_on_both_streaming_kernels(shape):
    ctx, _ = open_layer(shape, max_tokens=8192, max_batch=3)
    lens = [5000, 777, 9]
    q = make_query(shape, 3, seed=31)
    segs, qpos = [], []
    for b, T in enumerate(lens):
        K, V = make_kv(shape, T, seed=310 + b)
        cut = max(1, T - 100)
        segs.append([(K[:cut], V[:cut], 0), (K[cut:], V[cut:], cut)])
        qpos.append(T - 1)
    out = gpu_attention(ctx, shape, q, qpos, segs)
    attn_check(host_f64(out), oracle_attention(shape, q, qpos, segs))
    # one segment per sequence: identical bits
    segs1 = []
    for b, T in enumerate(lens):
        K, V = make_kv(shape, T, seed=310 + b)
        segs1.append([(K, V, 0)])
    out1 = gpu_attention(ctx, shape, q, qpos, segs1)
    assert torch.equal(out, out1)


@pytest.mark.parametrize("shape", [TINY_GQA, SMOLLM2_135M, GEMMA3_4B_LOCAL, QWEN3_4B, WIDE_SHAPES[1]], ids=lambda s: s.name)
def test_random_batches_of_random_layouts(shape):
    """Seeded random batches: lengths from 1 to 6000, one to four segments cut at random places, some
    with a gap or with keys beyond the query position, a random window override through the shape's own
    window -- every sequence against the oracle, and each sequence alone gives the bits it has in the batch."""
    rng = np.random.default_rng(1234 + shape.d_head + shape.n_q_heads)
    ctx, _ = open_layer(shape, max_tokens=8192, max_batch=7)
    for case in range(4):
        batch = int(rng.integers(1, 8))
        q = make_query(shape, batch, seed=500 + case)
        segs, qpos = [], []
        for b in range(batch):
            T = int(rng.choice([1, 2, 31, 33, 200, 1025, 2500, 6000]))
            K, V = make_kv(shape, T, seed=600 + 10 * case + b)
            n_cuts = int(rng.integers(0, 4))
            cuts = sorted(set(int(c) for c in rng.integers(1, T, size=n_cuts))) if T > 1 else []
            bounds = [0] + cuts + [T]
            gap = int(rng.integers(0, 2)) * 7  # shift everything after the first segment: a hole in the positions
            row = []
            for i in range(len(bounds) - 1):
                lo, hi = bounds[i], bounds[i + 1]
                row.append((K[lo:hi], V[lo:hi], lo + (gap if i > 0 else 0)))
            last_pos = T - 1 + (gap if len(bounds) > 2 else 0)
            qpos.append(max(0, last_pos - int(rng.integers(0, 3))))  # sometimes keys after the query
            segs.append(row)
        out = gpu_attention(ctx, shape, q, qpos, segs)
        ref = oracle_attention(shape, q, qpos, segs)
        for b in range(batch):
            attn_check(host_f64(out)[b], ref[b])
        b = int(rng.integers(0, batch))
        alone = gpu_attention(ctx, shape, q[b:b + 1], qpos[b:b + 1], segs[b:b + 1])
        assert torch.equal(alone[0], out[b])


@pytest.mark.parametrize("shape", [TINY_GQA, SMOLLM2_135M, GEMMA3_4B_GLOBAL, QWEN3_4B], ids=lambda s: s.name)
def test_segment_layout_does_not_change_the_bits(shape):
    """One stored segment (a full cache) and the same keys cut into recomputed / window / current
    segments must give identical output bits: the split over keys depends on positions only."""
    ctx, _ = open_layer(shape, max_tokens=4096)
    T = 2049
    K, V = make_kv(shape, T, seed=5)
    q = make_query(shape, 1, seed=5)
    base = host_bits(gpu_attention(ctx, shape, q, [T - 1], [[(K, V, 0)]]))
    for cuts in ([1793, 2048], [1, 2], [777], [64, 128, 2000]):
        edges = [0] + cuts + [T]
        segs = [[(K[a:b], V[a:b], a) for a, b in zip(edges[:-1], edges[1:])]]
        got = host_bits(gpu_attention(ctx, shape, q, [T - 1], segs))
        assert np.array_equal(got, base), cuts
    # order of the segment list is irrelevant as well
    segs = [[(K[2000:], V[2000:], 2000), (K[:2000], V[:2000], 0)]]
    assert np.array_equal(host_bits(gpu_attention(ctx, shape, q, [T - 1], segs)), base)


def test_no_visible_key_gives_zeros_and_single_key_gives_its_value():
    shape = TINY_GQA
    ctx, _ = open_layer(shape, max_tokens=1024)
    K, V = make_kv(shape, 4, seed=6)
    q = make_query(shape, 1, seed=6)
    # all keys lie after the query position
    out = gpu_attention(ctx, shape, q, [3], [[(K, V, 10)]])
    assert torch.all(out == 0)
    # no segment at all
    out = gpu_attention(ctx, shape, q, [3], [[]])
    assert torch.all(out == 0)
    # exactly one visible key: softmax weight 1, output == V (bit-exact, V is bf16 already)
    out = gpu_attention(ctx, shape, q, [10], [[(K, V, 10)]])
    g = shape.group
    got = host_bits(out)[0]
    for h in range(shape.n_q_heads):
        assert np.array_equal(got[h], V[0, h // g])


def test_argument_errors():
    shape = TINY_GQA
    ctx, _ = open_layer(shape, max_tokens=1024, max_batch=2)
    kdim = shape.n_kv_heads * shape.d_head
    K, V = make_kv(shape, 8, seed=7)
    k, v = dev(K), dev(V)
    q = dev(make_query(shape, 2, seed=7))
    out = torch.empty((2, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    ok = [(k, v, kdim, 0, 8)]
    for bad, status in (([(k, v, kdim - 8, 0, 8)], 1), ([(k, v, kdim + 4, 0, 8)], 3),
                        ([(k.data_ptr() + 2, v, kdim, 0, 8)], 3), ([(k, v, kdim, 0, 8), (k, v, kdim, 4, 8)], 1),
                        ([(k, v, kdim, -1, 8)], 1)):
        with pytest.raises(kvd.KvdError) as e:
            ctx.kvd_decode_attention(0, 1, q, [7], [bad], 0.0, out)
        assert e.value.status == status
    with pytest.raises(kvd.KvdError) as e:  # batch above max_batch
        ctx.kvd_decode_attention(0, 3, q, [7, 7, 7], [ok, ok, ok], 0.0, out)
    assert e.value.status == 4
    ctx.kvd_decode_attention(0, 2, q, [7, 7], [ok, ok], 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK


@pytest.mark.parametrize("shape", [GEMMA3_4B_LOCAL, QWEN3_4B], ids=lambda s: s.name)
def test_rows_of_one_sequence_with_their_own_causal_limit(shape):
    """kvd_decode_attention_rows: many query tokens of one sequence over shared segments, each seeing the keys up
    to its own position (and inside the window): every row must have the bits of a kvd_decode_attention call for
    that query alone, and follow the oracle called per row.  A small workspace forces several launches."""
    T, n_rows = 1500, 150
    ctx, _ = open_layer(shape, max_tokens=2048, max_batch=2)  # room for two sequences' partials: many launches
    kdim = shape.n_kv_heads * shape.d_head
    K, V = make_kv(shape, T, seed=5)
    cut = 900
    segs_bits = [(K[:cut], V[:cut], 0), (K[cut:], V[cut:], cut)]
    rng = np.random.default_rng(8)
    q_pos = sorted(rng.choice(np.arange(3, T + 40), n_rows, replace=False).tolist())  # some beyond the last key
    q_bits = make_query(shape, n_rows, seed=6)
    q = dev(q_bits)
    k0, v0, k1, v1 = dev(K[:cut]), dev(V[:cut]), dev(K[cut:]), dev(V[cut:])
    segs = [(k0, v0, kdim, 0, cut), (k1, v1, kdim, cut, T - cut)]
    out = torch.full((n_rows, shape.n_q_heads, shape.d_head), 9.0, dtype=torch.bfloat16, device="cuda")
    n0 = ctx.kvd_launch_count()
    ctx.kvd_decode_attention_rows(0, n_rows, q, q_pos, segs, 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert ctx.kvd_launch_count() - n0 > 2 * (n_rows // 64 + 1)  # the small workspace split the rows further
    one = torch.empty((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    for i in (0, 1, 63, 64, 77, n_rows - 1):
        ctx.kvd_decode_attention(0, 1, q[i:i + 1], [q_pos[i]], [segs], 0.0, one)
        assert torch.equal(one[0], out[i]), i
    sample = [0, 5, 64, 100, n_rows - 1]
    ref = oracle_attention(shape, q_bits[sample], [q_pos[i] for i in sample], [segs_bits] * len(sample))
    attn_check(host_f64(out[torch.tensor(sample).cuda()]), ref)
    ctx.close()


def test_a_sequences_bits_do_not_depend_on_the_rest_of_the_batch_or_the_kernel_variant():
    """One sequence of 4097 keys attended alone (260 CTAs: the streaming variant that issues the loads of both
    iterations at once) and as one of a batch of six (1,500 CTAs: the four-CTAs-per-SM variant): the same bits.  The
    split of a sequence is a function of its own visible range, and the two variants compute in the same order."""
    shape = GEMMA3_4B_GLOBAL
    lens = [4097, 1000, 4097, 2500, 65, 3333]
    ctx, _ = open_layer(shape, max_tokens=4200, max_batch=len(lens))
    kdim = shape.n_kv_heads * shape.d_head
    q_bits = make_query(shape, len(lens), seed=12)
    q = dev(q_bits)
    kv = [make_kv(shape, n, seed=30 + i) for i, n in enumerate(lens)]
    kd = [(dev(k), dev(v)) for k, v in kv]
    segs = [[(kd[i][0], kd[i][1], kdim, 0, n)] for i, n in enumerate(lens)]
    q_pos = [n - 1 for n in lens]
    out_b = torch.zeros((len(lens), shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_decode_attention(0, len(lens), q, q_pos, segs, 0.0, out_b)
    one = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    for i in range(len(lens)):
        ctx.kvd_decode_attention(0, 1, q[i:i + 1], [q_pos[i]], [segs[i]], 0.0, one)
        assert torch.equal(one[0], out_b[i]), i
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    ref = oracle_attention(shape, q_bits[:2], q_pos[:2], [[(kv[i][0], kv[i][1], 0)] for i in range(2)])
    attn_check(host_f64(out_b[:2]), ref)
    ctx.close()
