"""The whole path at a sequence length well above the benchmark's: 131072 tokens of the Gemma-3-4B-shaped global
layer in one sequence (671 MB of checkpoints, 2 x 268 MB of K/V, 512 row blocks, over a thousand tiles per
cluster walk).  K/V rows are sampled against the fp64 oracle (first and last rows, block edges, a seeded random
sample); the attention output over all 131072 keys is checked head group by head group against the oracle run
on the K/V the kernel produced (the attention kernels' own parity: its inputs are whatever K/V they are given)."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_19664_b200 as kvd
from kvd_synth import GEMMA3_4B_GLOBAL, bf16_to_f64, make_query, make_residuals
from gpu_util import dev, host_f64, kv_errors, open_layer, oracle_kv

pytestmark = pytest.mark.gpu


def test_one_sequence_of_131072_tokens():
    shape, T = GEMMA3_4B_GLOBAL, 131072
    ctx, w = open_layer(shape, max_tokens=T, with_store=True)
    kdim = shape.n_kv_heads * shape.d_head
    base = make_residuals(shape, 4096, seed=71, outliers=True)          # 4096 distinct rows, tiled 32 times
    X = np.tile(base, (T // 4096, 1))
    pos = np.arange(T, dtype=np.int32)
    x, p = dev(X), torch.from_numpy(pos).cuda()
    ctx.kvd_checkpoint_residual(0, 0, x, p, T)
    assert ctx.kvd_rows_stored(0, 0) == T
    K = torch.zeros((T, kdim), dtype=torch.bfloat16, device="cuda")
    V = torch.zeros_like(K)
    ctx.kvd_recompute_kv(0, None, None, T, K, V, kdim, seq=0, first_row=0)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    rows = np.unique(np.concatenate([np.random.default_rng(3).choice(T, 384, replace=False),
                                     [0, 1, 127, 128, 255, 256, 65535, 65536, T - 257, T - 256, T - 2, T - 1]]))
    Kr, Vr = oracle_kv(shape, w, X[rows], pos[rows])
    for name, g, r in (("K", host_f64(K[torch.from_numpy(rows).cuda()]), Kr.reshape(len(rows), kdim)),
                       ("V", host_f64(V[torch.from_numpy(rows).cuda()]), Vr.reshape(len(rows), kdim))):
        mx, rel = kv_errors(g, r)
        assert mx <= 2e-2 and rel <= 1e-2, (name, mx, rel)
    # identical residual rows at different positions: V does not depend on the position (Eq. 14)
    assert torch.equal(V[:4096], V[T - 4096:])
    q_bits = make_query(shape, 1, seed=72)
    out = torch.zeros((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
    ctx.kvd_decode_attention(0, 1, dev(q_bits), [T - 1], [[(K, V, kdim, 0, T)]], 0.0, out)
    assert ctx.kvd_poll_status() == kvd.KVD_OK
    got = host_f64(out)[0]
    qf = bf16_to_f64(q_bits[0])
    group = shape.n_q_heads // shape.n_kv_heads
    for h in range(shape.n_kv_heads):
        Kh = host_f64(K[:, h * shape.d_head:(h + 1) * shape.d_head].contiguous()).reshape(T, 1, shape.d_head)
        Vh = host_f64(V[:, h * shape.d_head:(h + 1) * shape.d_head].contiguous()).reshape(T, 1, shape.d_head)
        ref = oracle.decode_attention(qf[h * group:(h + 1) * group], T - 1, [(Kh, Vh, 0)], 1.0 / math.sqrt(shape.d_head), 0)
        d = got[h * group:(h + 1) * group] - ref
        assert np.linalg.norm(d) / np.linalg.norm(ref) <= 1e-2, h
        assert np.max(np.abs(d)) <= 1e-2 * np.max(np.abs(ref)) + 1e-30, h
