"""Pins for the oracle's Algorithm 1 (small stacks) and the cost model -- no GPU.

  * Proposition 3.2 / Table 2: K and V captured during the cached forward pass (Eq. 4-5, the stack's
    own Python restatement) equal the K and V rebuilt from the saved residual rows by the C
    reconstruction routine (Eq. 13-14), exactly, at sequence lengths 16..256: two separately written
    pieces of code that take the same operations in the same order.
  * Table 3 and the budget sweep of Section 5.6: greedy tokens under a bounded window with
    recomputation equal the full-cache tokens at every budget, 30 tokens.
  * Negative control: a bounded window *without* recomputation changes the logits.
  * Eq. 23-28 against the numbers the paper prints (tests/golden).
"""
import os

import numpy as np
import pytest

import oracle
from oracle import cost_model
from oracle.stack import OracleStack, weights_to_f64
from kvd_synth import S_GEMMA, S_QWEN, S_SMOL, bf16_to_f64, make_stack_weights, make_token_ids


def _weights(stack):
    return weights_to_f64(make_stack_weights(stack), bf16_to_f64)


@pytest.mark.parametrize("stack", [S_SMOL, S_GEMMA], ids=lambda s: s.name)
def test_reconstruction_identity_is_exact(stack):
    w = _weights(stack)
    lengths = (16, 32, 64, 128, 256)
    ids = make_token_ids(max(lengths), stack.vocab, seed=1)
    m = OracleStack(stack, w, "full")
    m.trace_kv = [[] for _ in range(stack.n_layers)]
    done = 0
    for T in lengths:
        for tok in ids[done:T]:
            m.step(int(tok))
        done = T
        for l in range(stack.n_layers):
            ls = stack.layer_shape(l)
            lw = w["layers"][l]
            X = np.stack(m.layers[l].rows[:T])
            K, V = oracle.recompute_kv(X, np.arange(T, dtype=np.int32), lw["gamma_in"], lw["w_kv"],
                                       stack.n_kv_heads, stack.d_head, stack.rms_eps, ls.rope_theta,
                                       lw.get("gamma_k") if stack.qk_norm else None, stack.rms_eps,
                                       stack.rope_style)
            Kc = np.stack([kv[0] for kv in m.trace_kv[l][:T]])
            Vc = np.stack([kv[1] for kv in m.trace_kv[l][:T]])
            assert np.max(np.abs(K - Kc)) == 0.0
            assert np.max(np.abs(V - Vc)) == 0.0


def test_window_relative_rotation_breaks_keys_not_values():
    # Eq. 16 / Table 2 last row: rotating a key by (j - w) instead of j changes K, never V
    stack = S_GEMMA
    w = _weights(stack)
    lw = w["layers"][0]
    ls = stack.layer_shape(0)
    X = bf16_to_f64(make_stack_weights(stack).embed[:8])
    pos = np.arange(40, 48, dtype=np.int32)
    args = (lw["gamma_in"], lw["w_kv"], stack.n_kv_heads, stack.d_head, stack.rms_eps, ls.rope_theta,
            lw["gamma_k"], stack.rms_eps)
    K_abs, V_abs = oracle.recompute_kv(X, pos, *args)
    K_rel, V_rel = oracle.recompute_kv(X, pos - 16, *args)
    assert np.max(np.abs(K_abs - K_rel)) > 1e-2
    assert np.array_equal(V_abs, V_rel)


@pytest.mark.parametrize("stack,ctx", [(S_GEMMA, 96), (S_QWEN, 64), (S_SMOL, 64)], ids=lambda x: getattr(x, "name", x))
def test_greedy_tokens_identical_at_every_budget(stack, ctx):
    w = _weights(stack)
    prompt = make_token_ids(ctx, stack.vocab, seed=2).tolist()
    ref_tokens, ref_logits = OracleStack(stack, w, "full").generate(prompt, 30)
    assert len(set(ref_tokens)) > 3, "degenerate generation: the test would prove nothing"
    for B in (0, 8, 16, 32, 64, 128, 256):
        toks, logits = OracleStack(stack, w, "kvdirect", B).generate(prompt, 30)
        assert toks == ref_tokens, f"budget {B}"
        for a, b in zip(logits, ref_logits):
            assert np.array_equal(a, b), f"budget {B}: logits differ"


@pytest.mark.parametrize("stack,ctx", [(S_GEMMA, 40), (S_QWEN, 32), (S_SMOL, 32)], ids=lambda x: getattr(x, "name", x))
def test_single_checkpoint_chained_recompute_is_exact(stack, ctx):
    """One checkpointed row per token (Eq. 24's d_hidden * b bytes): carrying the evicted tokens
    through the layers again every step reproduces the full-cache logits bit for bit (Prop. 3.2
    applied layer after layer), and what is held matches Eq. 28."""
    w = _weights(stack)
    prompt = make_token_ids(ctx, stack.vocab, seed=2).tolist()
    ref_tokens, ref_logits = OracleStack(stack, w, "full").generate(prompt, 12)
    assert len(set(ref_tokens)) > 2
    for B in (0, 8):
        m = OracleStack(stack, w, "chained", B)
        toks, logits = m.generate(prompt, 12)
        assert toks == ref_tokens, f"budget {B}"
        for a, b in zip(logits, ref_logits):
            assert np.array_equal(a, b), f"budget {B}: logits differ"
        assert m.replayed_rows > 0
        T = m.t
        assert len(m.rows0) == T and all(len(st.rows) == 0 for st in m.layers)
        assert all(len(st.win_k) == min(B, T) for st in m.layers)
        held = (len(m.rows0) - min(B, T)) * stack.d_hidden * 2 + \
            sum(len(st.win_k) for st in m.layers) * 2 * stack.n_kv_heads * stack.d_head * 2
        assert held == cost_model.total_memory(T, B, stack.n_layers, stack.n_kv_heads, stack.d_head, stack.d_hidden)


def test_window_without_recompute_is_not_lossless():
    # the comparison the paper draws (Section 5.6): dropping evicted tokens changes the output
    stack = S_QWEN
    w = _weights(stack)
    prompt = make_token_ids(64, stack.vocab, seed=2).tolist()
    full = OracleStack(stack, w, "full")
    for tok in prompt:
        a = full.step(tok)
    # "evict without recompute": a full-cache model whose cache is trimmed to the last 8 entries
    lossy = OracleStack(stack, w, "full")
    for tok in prompt:
        b = lossy.step(tok)
        for st in lossy.layers:
            while len(st.win_k) > 8:
                st.win_k.pop(0)
                st.win_v.pop(0)
                st.win_first += 1
    assert np.max(np.abs(a - b)) > 1e-6


# ------------------------------------------------------------------------------- cost model
def _rows(path):
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line.split()


def test_table1_memory_figures(golden_dir):
    n = 0
    for name, L, nkv, dh, d, kv_kb, res_kb, rho in _rows(os.path.join(golden_dir, "table1_memory.txt")):
        L, nkv, dh, d = int(L), int(nkv), int(dh), int(d)
        assert round(cost_model.kv_bytes_per_token(L, nkv, dh) / 1024.0, 1) == float(kv_kb), name
        assert round(cost_model.residual_bytes_per_token(d) / 1024.0, 1) == float(res_kb), name
        assert round(cost_model.compression_ratio(L, nkv, dh, d), 1) == float(rho), name
        n += 1
    assert n == 6


def test_gemma_worked_example(golden_dir):
    (kv, res, rho), = list(_rows(os.path.join(golden_dir, "gemma_worked_example.txt")))
    assert cost_model.kv_bytes_per_token(34, 4, 256, 2) == int(kv)
    assert cost_model.residual_bytes_per_token(2560, 2) == int(res)
    assert round(cost_model.compression_ratio(34, 4, 256, 2560), 1) == float(rho)


def test_cost_and_total_memory_forms():
    # Eq. 26: two projections of 2 N d_hidden d_head flops per KV head
    assert cost_model.recompute_flops(1, 4, 2560, 256) == 2 * (2 * 2560 * 256) * 4 == 10_485_760
    # Eq. 27
    assert cost_model.read_bytes(1, 4, 256, 2) == 4096
    # Eq. 28 limits: B = T is the unbounded cache, B = 0 is checkpoints only
    T, L, nkv, dh, d = 2048, 34, 4, 256, 2560
    assert cost_model.total_memory(T, T, L, nkv, dh, d) == T * cost_model.kv_bytes_per_token(L, nkv, dh)
    assert cost_model.total_memory(T, 0, L, nkv, dh, d) == T * cost_model.residual_bytes_per_token(d)
    # growth rate per token at fixed B is d_hidden * b, whatever the depth
    assert cost_model.total_memory(T + 1, 256, L, nkv, dh, d) - cost_model.total_memory(T, 256, L, nkv, dh, d) == d * 2
    # per-layer checkpoints cost L times more in the second term
    assert cost_model.per_layer_checkpoint_memory(T, 0, L, nkv, dh, d) == L * T * d * 2
