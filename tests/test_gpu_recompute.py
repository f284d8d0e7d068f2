"""GPU parity of kvd_recompute_kv / kvd_checkpoint_residual against the fp64 oracle (through the C ABI).

Tolerances (bf16 outputs against the fp64 oracle, per K and per V):
    max |gpu - oracle| <= 2e-2   and   ||gpu - oracle||_F / ||oracle||_F <= 1e-2.
Bit-identity tests compare raw bf16 bit patterns.
"""
import numpy as np
import pytest
import torch

import paper_2603_19664_b200 as kvd
from kvd_synth import (GEMMA3_4B_GLOBAL, GEMMA3_4B_LOCAL, QWEN3_4B, ROPE_HALF, SMOLLM2_135M, TINY_GQA, TINY_MHA,
                       make_residuals, with_style)
from gpu_util import dev, host_bits, host_f64, kv_errors, open_layer, oracle_kv

pytestmark = pytest.mark.gpu

MAX_ABS = 2e-2
REL_FRO = 1e-2


def run_gpu(ctx, shape, X_bits, pos, stride=None, sentinel_rows=0):
    n = X_bits.shape[0]
    kdim = shape.n_kv_heads * shape.d_head
    stride = stride or kdim
    x = dev(X_bits)
    p = torch.from_numpy(np.asarray(pos, np.int32)).cuda()
    k = torch.full((n + sentinel_rows, stride), -7.0, dtype=torch.bfloat16, device="cuda")
    v = torch.full((n + sentinel_rows, stride), -7.0, dtype=torch.bfloat16, device="cuda")
    ctx.kvd_recompute_kv(0, x, p, n, k, v, stride)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    return k, v


def check(shape, K, V, Kref, Vref, rows=None):
    kdim = shape.n_kv_heads * shape.d_head
    Kg = host_f64(K)[:, :kdim]
    Vg = host_f64(V)[:, :kdim]
    if rows is not None:
        Kg, Vg = Kg[rows], Vg[rows]
    Kr = Kref.reshape(Kref.shape[0], kdim)
    Vr = Vref.reshape(Vref.shape[0], kdim)
    for name, g, r in (("K", Kg, Kr), ("V", Vg, Vr)):
        mx, rel = kv_errors(g, r)
        assert mx <= MAX_ABS, f"{name}: max abs {mx}"
        assert rel <= REL_FRO, f"{name}: rel {rel}"


@pytest.mark.parametrize("shape", [TINY_GQA, TINY_MHA, SMOLLM2_135M], ids=lambda s: s.name)
@pytest.mark.parametrize("n", [1, 7, 127, 128, 129, 300])
def test_small_shapes_and_ragged_tiles(shape, n):
    ctx, w = open_layer(shape)
    X = make_residuals(shape, n, seed=n)
    pos = (np.arange(n) * 3 + 1) % 4096
    K, V = run_gpu(ctx, shape, X, pos)
    Kr, Vr = oracle_kv(shape, w, X, pos)
    check(shape, K, V, Kr, Vr)


def test_config1_smollm2_layer_full():
    # SmolLM2-135M layer, 512 checkpointed tokens at positions 0..511
    shape = SMOLLM2_135M
    ctx, w = open_layer(shape)
    X = make_residuals(shape, 512, seed=1)
    pos = np.arange(512)
    K, V = run_gpu(ctx, shape, X, pos, sentinel_rows=4)
    Kr, Vr = oracle_kv(shape, w, X, pos)
    check(shape, K[:512], V[:512], Kr, Vr)
    # guard rows behind the output stay untouched
    assert torch.all(K[512:] == -7.0) and torch.all(V[512:] == -7.0)


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, GEMMA3_4B_LOCAL], ids=lambda s: s.name)
def test_config2_gemma_layer_t4096_sampled(shape):
    # full-size launch (T = 4096, outlier channels); the oracle checks the first and last row of
    # every 128-row tile class plus a random sample
    T = 4096
    ctx, w = open_layer(shape, max_tokens=32768)
    X = make_residuals(shape, T, seed=2, outliers=True)
    pos = np.arange(T)
    K, V = run_gpu(ctx, shape, X, pos)
    rng = np.random.default_rng(0)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 129, 2047, 2048, T - 129, T - 128, T - 1],
                                     rng.choice(T, 150, replace=False)]))
    Kr, Vr = oracle_kv(shape, w, X[rows], pos[rows])
    check(shape, K, V, Kr, Vr, rows=rows)


def test_qwen3_shape_two_heads_per_tile_and_large_positions():
    shape = QWEN3_4B
    ctx, w = open_layer(shape, max_tokens=32768)
    n = 333
    X = make_residuals(shape, n, seed=3)
    pos = np.concatenate([np.arange(32768 - 200, 32768), np.arange(0, n - 200)])
    K, V = run_gpu(ctx, shape, X, pos)
    rows = np.arange(0, n, 3)
    Kr, Vr = oracle_kv(shape, w, X[rows], pos[rows])
    check(shape, K, V, Kr, Vr, rows=rows)


@pytest.mark.parametrize("shape", [TINY_GQA, SMOLLM2_135M, GEMMA3_4B_GLOBAL], ids=lambda s: s.name)
def test_half_rotation_style(shape):
    shape = with_style(shape, ROPE_HALF)
    ctx, w = open_layer(shape, max_tokens=8192)
    n = 140
    X = make_residuals(shape, n, seed=4)
    pos = np.arange(n) * 37 % 8192
    K, V = run_gpu(ctx, shape, X, pos)
    rows = np.arange(0, n, 2)
    Kr, Vr = oracle_kv(shape, w, X[rows], pos[rows])
    check(shape, K, V, Kr, Vr, rows=rows)


def test_fused_output_buffer_with_row_stride():
    # K and V side by side in one [n, 2*kdim] buffer
    shape = TINY_GQA
    ctx, w = open_layer(shape)
    n, kdim = 70, shape.n_kv_heads * shape.d_head
    X = make_residuals(shape, n, seed=5)
    pos = np.arange(n)
    buf = torch.zeros((n, 2 * kdim), dtype=torch.bfloat16, device="cuda")
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    ctx._check(ctx._lib.kvd_recompute_kv(ctx._h, 0, x.data_ptr(), p.data_ptr(), n, 0, 0, buf.data_ptr(),
                                         buf.data_ptr() + kdim * 2, 2 * kdim, None), "kvd_recompute_kv")
    torch.cuda.synchronize()
    Kr, Vr = oracle_kv(shape, w, X, pos)
    check(shape, buf[:, :kdim], buf[:, kdim:], Kr, Vr)


@pytest.mark.parametrize("shape", [TINY_GQA, SMOLLM2_135M, GEMMA3_4B_GLOBAL], ids=lambda s: s.name)
def test_recompute_is_bit_identical_to_first_pass(shape):
    """Proposition 3.2 on the GPU: a row's K/V bits do not depend on the batch it is computed in."""
    ctx, w = open_layer(shape, max_tokens=8192)
    T = 4096 if shape is GEMMA3_4B_GLOBAL else 600
    X = make_residuals(shape, T, seed=6, outliers=shape is GEMMA3_4B_GLOBAL)
    pos = np.arange(T) + 11
    K, V = run_gpu(ctx, shape, X, pos)
    Kb, Vb = host_bits(K), host_bits(V)
    # first pass: one token at a time (M = 1), as a decode step produces K_t, V_t
    for m in (0, 1, 127, 128, T - 1):
        k1, v1 = run_gpu(ctx, shape, X[m:m + 1], pos[m:m + 1])
        assert np.array_equal(host_bits(k1)[0], Kb[m]) and np.array_equal(host_bits(v1)[0], Vb[m])
    # the same rows at other batch positions and batch sizes
    for start, n in ((5, 7), (100, 128), (77, 129), (T - 130, 130)):
        k2, v2 = run_gpu(ctx, shape, X[start:start + n], pos[start:start + n])
        assert np.array_equal(host_bits(k2), Kb[start:start + n])
        assert np.array_equal(host_bits(v2), Vb[start:start + n])
    perm = np.random.default_rng(1).permutation(T)[:257]
    k3, v3 = run_gpu(ctx, shape, X[perm], pos[perm])
    assert np.array_equal(host_bits(k3), Kb[perm]) and np.array_equal(host_bits(v3), Vb[perm])
    # run-to-run determinism
    K2, V2 = run_gpu(ctx, shape, X, pos)
    assert np.array_equal(host_bits(K2), Kb) and np.array_equal(host_bits(V2), Vb)


def test_checkpoint_store_roundtrip_and_recompute_from_store():
    shape = SMOLLM2_135M
    ctx, w = open_layer(shape, max_tokens=512, max_seqs=2, with_store=True)
    kdim = shape.n_kv_heads * shape.d_head
    X = make_residuals(shape, 300, seed=7)
    pos = np.arange(300) + 5
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    # append in two pieces to sequence 1, something else to sequence 0
    ctx.kvd_checkpoint_residual(1, 0, x[:100], p[:100], 100)
    ctx.kvd_checkpoint_residual(0, 0, x[200:], p[200:], 100)
    ctx.kvd_checkpoint_residual(1, 0, x[100:], p[100:], 200)
    assert ctx.kvd_rows_stored(0, 1) == 300 and ctx.kvd_rows_stored(0, 0) == 100
    stats = ctx.kvd_memory_stats()
    assert stats["checkpoint_bytes_used"] == 400 * (shape.d_hidden * 2 + 8)
    assert stats["eq24_residual_bytes_per_token"] == shape.d_hidden * 2
    K, V = run_gpu(ctx, shape, X, pos)
    k = torch.zeros((250, kdim), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros_like(k)
    ctx.kvd_recompute_kv(0, None, None, 250, k, v, kdim, seq=1, first_row=50)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert torch.equal(k, K[50:300]) and torch.equal(v, V[50:300])
    Kr, Vr = oracle_kv(shape, w, X[50:300], pos[50:300])
    check(shape, k, v, Kr, Vr)
    # capacity and state errors are reported, nothing is launched
    with pytest.raises(kvd.KvdError) as e:
        ctx.kvd_recompute_kv(0, None, None, 10, k, v, kdim, seq=0, first_row=95)
    assert e.value.status == 4
    with pytest.raises(kvd.KvdError) as e:
        ctx.kvd_checkpoint_residual(1, 0, x, p, 300)
    assert e.value.status == 4
    ctx.kvd_reset_sequence(1)
    assert ctx.kvd_rows_stored(0, 1) == 0


def test_row_statistic_kept_in_the_store_is_the_sum_of_squares():
    """The third region of the arena (rows, positions, sums of squares, each starting at a 256-byte
    multiple) holds the RMSNorm statistic of Eq. 2 for every checkpointed row."""
    shape = GEMMA3_4B_GLOBAL
    max_tokens, n = 384, 300
    desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                         shape.qk_norm, shape.rms_eps, shape.rope_style, 2, max_tokens, 1)
    ctx = kvd.Kvd(desc)
    arena = torch.zeros(kvd.kvd_store_bytes(desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store(arena, 1)
    X = make_residuals(shape, n, seed=17, outliers=True)
    pos = np.arange(n) + 3
    x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
    ctx.kvd_checkpoint_residual(1, 0, x[:7], p[:7], 7)      # two appends to sequence slot 1
    ctx.kvd_checkpoint_residual(1, 0, x[7:], p[7:], n - 7)
    torch.cuda.synchronize()
    slots = 2 * max_tokens
    ru = lambda b: (b + 255) // 256 * 256
    rows_bytes, pos_bytes = ru(slots * shape.d_hidden * 2), ru(slots * 4)
    assert arena.numel() == rows_bytes + 2 * pos_bytes
    a = arena.cpu().numpy()
    got_rows = a[:rows_bytes].view(np.uint16).reshape(-1, shape.d_hidden)[max_tokens:max_tokens + n]
    got_pos = a[rows_bytes:rows_bytes + pos_bytes].view(np.int32)[max_tokens:max_tokens + n]
    got_ss = a[rows_bytes + pos_bytes:].view(np.float32)[max_tokens:max_tokens + n]
    assert np.array_equal(got_rows, X) and np.array_equal(got_pos, pos)
    from kvd_synth import bf16_to_f64
    ref = np.sum(bf16_to_f64(X) ** 2, axis=1)
    assert np.max(np.abs(got_ss - ref) / ref) < 1e-6   # fp32 accumulation of 2560 exact squares


@pytest.mark.parametrize("shape", [SMOLLM2_135M, GEMMA3_4B_GLOBAL], ids=lambda s: s.name)
def test_output_bits_do_not_depend_on_output_alignment_or_row_count_path(shape):
    """32-byte-aligned outputs take 32-byte stores, others 16-byte stores; 1..64 caller rows have their
    statistics taken inside the kernel, more by a kernel of their own: the bits must not change."""
    ctx, w = open_layer(shape, max_tokens=1024)
    kdim = shape.n_kv_heads * shape.d_head
    T = 300
    X = make_residuals(shape, T, seed=18, outliers=True)
    pos = np.arange(T) + 40
    K, V = run_gpu(ctx, shape, X, pos)
    Kb, Vb = host_bits(K), host_bits(V)
    for n in (1, 3, 33, 64, 65, 129, T):
        x, p = dev(X[:n]), torch.from_numpy(pos[:n].astype(np.int32)).cuda()
        stride = kdim + 8                       # rows 16-byte but not 32-byte aligned
        kbuf = torch.full((n * stride + 8,), -7.0, dtype=torch.bfloat16, device="cuda")
        vbuf = torch.full((n * stride + 8,), -7.0, dtype=torch.bfloat16, device="cuda")
        ctx._check(ctx._lib.kvd_recompute_kv(ctx._h, 0, x.data_ptr(), p.data_ptr(), n, 0, 0, kbuf.data_ptr() + 16,
                                             vbuf.data_ptr() + 16, stride, None), "kvd_recompute_kv")
        assert ctx.kvd_poll_status() == kvd.KVD_OK
        k = host_bits(kbuf[8:].view(n, stride))
        v = host_bits(vbuf[8:].view(n, stride))
        assert np.array_equal(k[:, :kdim], Kb[:n]) and np.array_equal(v[:, :kdim], Vb[:n]), n
        pad = host_bits(torch.full((1,), -7.0, dtype=torch.bfloat16))[0]
        assert np.all(k[:, kdim:] == pad) and np.all(v[:, kdim:] == pad)   # nothing written between rows
        assert host_bits(kbuf[:8]).tolist() == [pad] * 8


@pytest.mark.parametrize("shape", [SMOLLM2_135M, GEMMA3_4B_GLOBAL], ids=lambda s: s.name)
def test_step_call_matches_separate_calls_bit_for_bit(shape):
    """kvd_recompute_kv_step: ranges of three sequences (ragged, non-zero first rows, one empty) plus
    new-token rows in one launch == one kvd_recompute_kv call per source, and within tolerance of
    the oracle; rows after each range's end are left untouched."""
    ctx, w = open_layer(shape, max_tokens=1024, max_seqs=4, with_store=True)
    kdim = shape.n_kv_heads * shape.d_head
    n_seq = [700, 300, 0, 513]
    Xs, Ps = [], []
    for s, n in enumerate(n_seq):
        X = make_residuals(shape, max(n, 1), seed=40 + s)[:n]
        pos = (np.arange(n) + 3 * s).astype(np.int32)
        Xs.append(X)
        Ps.append(pos)
        if n:
            ctx.kvd_checkpoint_residual(s, 0, dev(X), torch.from_numpy(pos).cuda(), n)
    ranges_spec = [(0, 37, 600), (1, 0, 300), (2, 0, 0), (3, 256, 257)]
    Xn = make_residuals(shape, 3, seed=50)
    pn = np.array([700, 303, 519], np.int32)
    xn, pnd = dev(Xn), torch.from_numpy(pn).cuda()

    def outputs():
        ks = [torch.full((n + 2, kdim), -7.0, dtype=torch.bfloat16, device="cuda") for (_, _, n) in ranges_spec]
        vs = [torch.full((n + 2, kdim), -7.0, dtype=torch.bfloat16, device="cuda") for (_, _, n) in ranges_spec]
        kn = torch.full((3 + 2, kdim), -7.0, dtype=torch.bfloat16, device="cuda")
        vn = torch.full((3 + 2, kdim), -7.0, dtype=torch.bfloat16, device="cuda")
        return ks, vs, kn, vn

    ks, vs, kn, vn = outputs()
    launches = ctx.kvd_launch_count()
    ctx.kvd_recompute_kv_step(0, [(s, f, n, ks[i], vs[i]) for i, (s, f, n) in enumerate(ranges_spec)], xn, pnd, 3,
                              kn, vn, kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    assert ctx.kvd_launch_count() == launches + 1
    ks2, vs2, kn2, vn2 = outputs()
    for i, (s, f, n) in enumerate(ranges_spec):
        ctx.kvd_recompute_kv(0, None, None, n, ks2[i], vs2[i], kdim, seq=s, first_row=f)
    ctx.kvd_recompute_kv(0, xn, pnd, 3, kn2, vn2, kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    for a, b in zip(ks + vs + [kn, vn], ks2 + vs2 + [kn2, vn2]):
        assert torch.equal(a, b)
    sentinel = host_bits(torch.full((1,), -7.0, dtype=torch.bfloat16))[0]
    for i, (s, f, n) in enumerate(ranges_spec):
        assert np.all(host_bits(ks[i])[n:] == sentinel) and np.all(host_bits(vs[i])[n:] == sentinel)
        if n:
            Kr, Vr = oracle_kv(shape, w, Xs[s][f:f + n], Ps[s][f:f + n])
            check(shape, ks[i][:n], vs[i][:n], Kr, Vr)
    assert np.all(host_bits(kn)[3:] == sentinel) and np.all(host_bits(vn)[3:] == sentinel)
    Kr, Vr = oracle_kv(shape, w, Xn, pn)
    check(shape, kn[:3], vn[:3], Kr, Vr)
    # ranges only; rows only
    ks3, vs3, kn3, vn3 = outputs()
    ctx.kvd_recompute_kv_step(0, [(s, f, n, ks3[i], vs3[i]) for i, (s, f, n) in enumerate(ranges_spec)], None, None, 0,
                              None, None, kdim)
    ctx.kvd_recompute_kv_step(0, [], xn, pnd, 3, kn3, vn3, kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    for a, b in zip(ks + vs + [kn, vn], ks3 + vs3 + [kn3, vn3]):
        assert torch.equal(a, b)
    # a range past the stored rows rejects the whole call before anything is launched
    launches = ctx.kvd_launch_count()
    with pytest.raises(kvd.KvdError) as e:
        ctx.kvd_recompute_kv_step(0, [(0, 0, 10, ks[0], vs[0]), (1, 290, 11, ks[1], vs[1])], xn, pnd, 3, kn, vn, kdim)
    assert e.value.status == 4
    with pytest.raises(kvd.KvdError) as e:
        ctx.kvd_recompute_kv_step(0, [(0, 0, 1, ks[0], vs[0])] * 65, None, None, 0, None, None, kdim)
    assert e.value.status == 1
    assert ctx.kvd_launch_count() == launches


def test_step_call_with_64_sequences():
    """A batch of 64 sequences with different evicted lengths and 64 new tokens in one launch."""
    shape = TINY_GQA
    ctx, w = open_layer(shape, max_tokens=640, max_seqs=64, max_batch=64, with_store=True)
    kdim = shape.n_kv_heads * shape.d_head
    rng = np.random.default_rng(77)
    lens = rng.integers(1, 600, size=64)
    ranges, refs = [], []
    for s in range(64):
        n = int(lens[s])
        X = make_residuals(shape, n, seed=900 + s)
        pos = np.arange(n, dtype=np.int32)
        ctx.kvd_checkpoint_residual(s, 0, dev(X), torch.from_numpy(pos).cuda(), n)
        k = torch.zeros((n, kdim), dtype=torch.bfloat16, device="cuda")
        v = torch.zeros_like(k)
        ranges.append((s, 0, n, k, v))
        refs.append((X, pos))
    Xn = make_residuals(shape, 64, seed=990)
    pn = lens.astype(np.int32)
    kn = torch.zeros((64, kdim), dtype=torch.bfloat16, device="cuda")
    vn = torch.zeros_like(kn)
    ctx.kvd_recompute_kv_step(0, ranges, dev(Xn), torch.from_numpy(pn).cuda(), 64, kn, vn, kdim)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    for s in (0, 1, 17, 40, 63):
        Kr, Vr = oracle_kv(shape, w, *refs[s])
        check(shape, ranges[s][3], ranges[s][4], Kr, Vr)
    Kr, Vr = oracle_kv(shape, w, Xn, pn)
    check(shape, kn, vn, Kr, Vr)
    # every range equals the single-source call
    for s in (5, 33, 62):
        n = int(lens[s])
        k = torch.zeros((n, kdim), dtype=torch.bfloat16, device="cuda")
        v = torch.zeros_like(k)
        ctx.kvd_recompute_kv(0, None, None, n, k, v, kdim, seq=s, first_row=0)
        assert torch.equal(k, ranges[s][3]) and torch.equal(v, ranges[s][4])


def test_step_sequence_in_a_cuda_graph_on_a_side_stream_matches_eager():
    """checkpoint -> recompute (store range + new token) -> attention, captured into a CUDA graph on a
    non-default stream (the kernels are programmatic dependents of one another) and replayed several
    times, gives the bits of the eager sequence on the default stream."""
    shape = GEMMA3_4B_GLOBAL
    T = 600
    ctx, w = open_layer(shape, max_tokens=1024, max_seqs=2, with_store=True)
    kdim = shape.n_kv_heads * shape.d_head
    X = dev(make_residuals(shape, T + 1, seed=61, outliers=True))
    pos = torch.arange(T + 1, dtype=torch.int32, device="cuda")
    q = torch.randn((1, shape.n_q_heads, shape.d_head), device="cuda").to(torch.bfloat16)

    def sequence(seq, K, V, out):
        ctx.kvd_reset_sequence(seq)
        ctx.kvd_checkpoint_residual(seq, 0, X, pos, T)
        ctx.kvd_recompute_kv_step(0, [(seq, 0, T, K, V)], X[T:], pos[T:], 1, K[T:], V[T:], kdim)
        ctx.kvd_decode_attention(0, 1, q, [T], [[(K, V, kdim, 0, T), (K[T:], V[T:], kdim, T, 1)]], 0.0, out)

    def buffers():
        return (torch.zeros((T + 1, kdim), dtype=torch.bfloat16, device="cuda"),
                torch.zeros((T + 1, kdim), dtype=torch.bfloat16, device="cuda"),
                torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda"))

    K0, V0, o0 = buffers()
    sequence(0, K0, V0, o0)
    torch.cuda.synchronize()
    K1, V1, o1 = buffers()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        sequence(1, K1, V1, o1)  # warm-up on the capture stream
    side.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        sequence(1, K1, V1, o1)
    for _ in range(3):
        K1.zero_(); V1.zero_(); o1.zero_()
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(K1, K0) and torch.equal(V1, V0) and torch.equal(o1, o0)
    assert ctx.kvd_poll_status() == kvd.KVD_OK


def test_argument_errors_and_position_flag():
    shape = TINY_GQA
    ctx, w = open_layer(shape, max_tokens=1024)
    kdim = shape.n_kv_heads * shape.d_head
    X = make_residuals(shape, 16, seed=8)
    x = dev(X)
    p = torch.arange(16, dtype=torch.int32, device="cuda")
    k = torch.zeros((16, kdim), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros_like(k)
    lib, h = ctx._lib, ctx._h
    assert lib.kvd_recompute_kv(h, 0, x.data_ptr() + 2, p.data_ptr(), 4, 0, 0, k.data_ptr(), v.data_ptr(), kdim, None) == 3
    assert lib.kvd_recompute_kv(h, 0, x.data_ptr(), p.data_ptr(), 4, 0, 0, k.data_ptr(), v.data_ptr(), kdim - 8, None) == 1
    assert lib.kvd_recompute_kv(h, 0, x.data_ptr(), p.data_ptr(), 4, 0, 0, k.data_ptr(), v.data_ptr(), kdim + 4, None) == 3
    assert lib.kvd_recompute_kv(h, 3, x.data_ptr(), p.data_ptr(), 4, 0, 0, k.data_ptr(), v.data_ptr(), kdim, None) == 1
    assert lib.kvd_recompute_kv(h, 0, x.data_ptr(), None, 4, 0, 0, k.data_ptr(), v.data_ptr(), kdim, None) == 1
    assert lib.kvd_recompute_kv(h, 0, x.data_ptr(), p.data_ptr(), 0, 0, 0, None, None, kdim, None) == 0  # n = 0: no-op
    # a position outside [0, max_tokens) is flagged, clamped, and faults nothing
    bad = p.clone()
    bad[3] = 5000
    bad[9] = -2
    ctx.kvd_recompute_kv(0, x, bad, 16, k, v, kdim)
    assert ctx.kvd_poll_status() == 9
    assert ctx.kvd_poll_status() == kvd.KVD_OK  # the flag is cleared by the read
    assert ctx.kvd_launch_count() >= 2


def test_bounded_wait_expires_and_is_reported_without_harming_the_device():
    """Failure detection: a wait that nothing satisfies gives up after its limit, the kernel returns,
    kvd_poll_status says KVD_ERR_TIMEOUT, and the context keeps working."""
    shape = TINY_GQA
    ctx, w = open_layer(shape)
    ctx.kvd_selftest_wait_timeout(5)
    assert ctx.kvd_poll_status() == 8  # KVD_ERR_TIMEOUT
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    X = make_residuals(shape, 40, seed=9)
    pos = np.arange(40)
    K, V = run_gpu(ctx, shape, X, pos)
    Kr, Vr = oracle_kv(shape, w, X, pos)
    check(shape, K, V, Kr, Vr)
    # the trace hook records a timeline and does not change results
    tr = torch.zeros((148, 8, 16), dtype=torch.int64, device="cuda")
    ctx.kvd_set_trace(tr)
    K2, V2 = run_gpu(ctx, shape, X, pos)
    ctx.kvd_set_trace(None)
    assert torch.equal(K, K2) and torch.equal(V, V2)
    t = tr.cpu().numpy()
    assert t[0, 0, 5] > t[0, 0, 4] > 0 and t[0, 0, 7] > t[0, 0, 6] > 0  # MMA and epilogue intervals of tile 0


@pytest.mark.parametrize("shape", [GEMMA3_4B_GLOBAL, SMOLLM2_135M], ids=lambda s: s.name)
def test_decode_step_kv_equals_the_separate_calls_bit_for_bit(shape):
    """kvd_decode_step_kv = STORE_RESIDUAL of the new rows + RECOMPUTE_KV of the evicted ranges + (K_t, V_t), one
    launch: the store (rows, positions, statistics, counts), the recomputed K/V and the new tokens' K/V written
    with a stride of their own must equal what kvd_checkpoint_residual_step + kvd_recompute_kv_step leave."""
    batch, T, max_tokens = 5, 300, 512
    kdim = shape.n_kv_heads * shape.d_head
    desc_args = dict(max_tokens=max_tokens, max_batch=batch, max_seqs=batch, with_store=True)
    ctx_a, w = open_layer(shape, **desc_args)
    ctx_b, _ = open_layer(shape, **desc_args)
    arena_a, arena_b = ctx_a._keep[-1], ctx_b._keep[-1]
    arena_a.zero_()
    arena_b.zero_()
    X = dev(make_residuals(shape, T + batch, seed=31, outliers=True))
    pos = torch.arange(T, dtype=torch.int32, device="cuda")
    for b in range(batch):
        rows = torch.roll(X[:T], shifts=-7 * b, dims=0).contiguous()
        for c in (ctx_a, ctx_b):
            c.kvd_checkpoint_residual(b, 0, rows, pos, T - b)   # ragged: sequence b holds T - b rows
    x_new = X[T:T + batch].contiguous()
    p_new = torch.tensor([T - b for b in range(batch)], dtype=torch.int32, device="cuda")
    n_old = [T - b - 40 for b in range(batch)]
    ko = [torch.zeros((T, kdim), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    vo = [torch.zeros((T, kdim), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    # (a) separate calls, contiguous K_t/V_t
    ka, va = torch.zeros((batch, kdim), dtype=torch.bfloat16, device="cuda"), torch.zeros((batch, kdim), dtype=torch.bfloat16, device="cuda")
    ctx_a.kvd_checkpoint_residual_step(0, list(range(batch)), x_new, p_new)
    ctx_a.kvd_recompute_kv_step(0, [(b, 3, n_old[b], ko[0][3:], vo[0][3:]) for b in range(1)] +
                                [(b, 0, 0, None, None) for b in range(1, batch)], x_new, p_new, batch, ka, va, kdim)
    # (b) one launch; K_t/V_t scattered into a [batch][max_tokens][kdim] cache at each sequence's position 9
    cache_k = torch.full((batch, max_tokens, kdim), 7.0, dtype=torch.bfloat16, device="cuda")
    cache_v = torch.full_like(cache_k, 7.0)
    n0 = ctx_b.kvd_launch_count()
    ctx_b.kvd_decode_step_kv(0, [(0, 3, n_old[0], ko[1][3:], vo[1][3:])], kdim, x_new, p_new, batch, list(range(batch)),
                             cache_k[0, 9], cache_v[0, 9], max_tokens * kdim)
    assert ctx_b.kvd_launch_count() - n0 == 1
    assert ctx_a.kvd_poll_status() == kvd.KVD_OK and ctx_b.kvd_poll_status() == kvd.KVD_OK
    assert torch.equal(arena_a, arena_b), "store contents differ"
    for b in range(batch):
        assert ctx_a.kvd_rows_stored(0, b) == ctx_b.kvd_rows_stored(0, b) == T - b + 1
    assert torch.equal(ko[0], ko[1]) and torch.equal(vo[0], vo[1])
    assert torch.equal(cache_k[:, 9], ka) and torch.equal(cache_v[:, 9], va)
    untouched = torch.ones((max_tokens,), dtype=torch.bool, device="cuda")
    untouched[9] = False
    assert torch.all(cache_k[:, untouched] == 7.0) and torch.all(cache_v[:, untouched] == 7.0)
    # the appended rows can be recomputed from the store like any other (same bits as from the caller's buffer)
    k2, v2 = torch.zeros((1, kdim), dtype=torch.bfloat16, device="cuda"), torch.zeros((1, kdim), dtype=torch.bfloat16, device="cuda")
    for b in (0, batch - 1):
        ctx_b.kvd_recompute_kv(0, None, None, 1, k2, v2, kdim, seq=b, first_row=T - b)
        assert torch.equal(k2[0], ka[b]) and torch.equal(v2[0], va[b])
    # limits: more than 64 appended rows, a full sequence, a bad slot -- nothing stored
    before = [ctx_b.kvd_rows_stored(0, b) for b in range(batch)]
    big = torch.zeros((65, shape.d_hidden), dtype=torch.bfloat16, device="cuda")
    pb = torch.zeros((65,), dtype=torch.int32, device="cuda")
    kb, vb = torch.zeros((65, kdim), dtype=torch.bfloat16, device="cuda"), torch.zeros((65, kdim), dtype=torch.bfloat16, device="cuda")
    for seqs, n, status in (([0] * 65, 65, 4), ([batch], 1, 1), ([0] * 64, 64, 4 if before[0] + 64 > max_tokens else 0)):
        try:
            ctx_b.kvd_decode_step_kv(0, [], kdim, big, pb, n, seqs, kb, vb, kdim)
            got = 0
        except kvd.KvdError as e:
            got = e.status
        assert got == status, (seqs[:2], n, got)
    if before[0] + 64 > max_tokens:
        assert [ctx_b.kvd_rows_stored(0, b) for b in range(batch)] == before
    ctx_a.close()
    ctx_b.close()
