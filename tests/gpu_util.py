"""Helpers shared by the GPU tests: move seeded inputs to the device and open a library context."""
import numpy as np
import torch

import paper_2603_19664_b200 as kvd
from kvd_synth import bf16_to_f64, make_layer_weights


def dev(bits: np.ndarray) -> torch.Tensor:
    """bf16 bit patterns (uint16) -> bf16 tensor on the GPU."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def host_f64(t: torch.Tensor) -> np.ndarray:
    """bf16 device tensor -> float64 numpy (exact)."""
    return bf16_to_f64(t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16))


def host_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def open_layer(shape, max_tokens=4096, max_batch=1, max_seqs=1, layer_seed=0, with_store=False, weights=None):
    """One-layer context for a kvd_synth.LayerShape; returns (ctx, weights, keepalive tensors)."""
    w = weights if weights is not None else make_layer_weights(shape, layer_seed)
    desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                         shape.qk_norm, shape.rms_eps, shape.rope_style, max_seqs, max_tokens, max_batch)
    ctx = kvd.Kvd(desc)
    t_w = dev(w.w_kv)
    t_g = dev(w.gamma_in)
    t_gk = dev(w.gamma_k) if w.gamma_k is not None else None
    ctx.kvd_set_layer(0, t_w, t_g, t_gk, shape.rope_theta, shape.sliding_window)
    ws = torch.empty(kvd.kvd_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_workspace(ws)
    if with_store:
        arena = torch.empty(kvd.kvd_store_bytes(desc, 1), dtype=torch.uint8, device="cuda")
        ctx.kvd_attach_store(arena, 1)
    return ctx, w


def oracle_kv(shape, w, X_bits, pos):
    import oracle
    return oracle.recompute_kv(bf16_to_f64(X_bits), np.asarray(pos, np.int32), bf16_to_f64(w.gamma_in),
                               bf16_to_f64(w.w_kv), shape.n_kv_heads, shape.d_head, shape.rms_eps, shape.rope_theta,
                               bf16_to_f64(w.gamma_k) if w.gamma_k is not None else None, shape.rms_eps,
                               shape.rope_style)


def kv_errors(got_f64: np.ndarray, ref: np.ndarray):
    """(max abs error, relative Frobenius error)."""
    d = got_f64 - ref
    return float(np.max(np.abs(d))), float(np.linalg.norm(d) / max(np.linalg.norm(ref), 1e-300))
