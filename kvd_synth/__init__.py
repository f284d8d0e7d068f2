"""Seeded synthetic inputs for the KV-Direct hot path.

This module only *generates data*: shapes, random weights, residual rows, queries,
token ids.  It contains none of the method's arithmetic (no normalisation, projection,
rotation or attention), so both the CPU oracle's tests and the CUDA path's tests can
import it without sharing any computation.

Every array is drawn in float32 from ``numpy.random.Generator(PCG64(seed))`` and then
rounded to bfloat16 (round-to-nearest-even).  Arrays are returned as ``uint16`` bit
patterns; ``bf16_to_f64`` widens them exactly for the oracle, and the GPU side views the
same bits as ``torch.bfloat16``.

Shapes follow the models listed in the paper's Table 1 (SmolLM2-135M, Gemma-3-4B) plus the
Qwen3-4B shape used for the long-context case.  Weights are N(0, 0.02), residual rows are
N(0, 1); the Gemma-shaped case multiplies 1 % of the channels by 20 to mimic the outlier
channels of real residual streams.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional

import numpy as np

ROPE_INTERLEAVED = 0  # consecutive pairs (2i, 2i+1): the pairing of the paper's Eq. 11-12
ROPE_HALF = 1  # pairs (i, i + d_head/2)

# seed bases, one family per kind of tensor
SEED_WEIGHTS = 1000
SEED_NORMS = 2000
SEED_RESIDUALS = 3000
SEED_QUERY = 4000
SEED_TOKENS = 5000
SEED_OUTLIERS = 6000
SEED_KV = 7000


# --------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even) and return the uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    nan = np.isnan(a)
    rounding = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    out = ((u + rounding) >> np.uint32(16)).astype(np.uint16)
    if nan.any():
        out = np.where(nan, np.uint16(0x7FC0), out)
    return out


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to float32 (exact)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to float64 (exact)."""
    return bf16_to_f32(bits).astype(np.float64)


def _normal_bf16(rng: np.random.Generator, shape, std: float, mean: float = 0.0) -> np.ndarray:
    a = rng.standard_normal(size=shape, dtype=np.float32) * np.float32(std) + np.float32(mean)
    return f32_to_bf16_bits(a)


# --------------------------------------------------------------------------- shapes
@dataclass(frozen=True)
class LayerShape:
    """Dimensions and constants of one decoder layer's attention block."""

    name: str
    d_hidden: int
    n_q_heads: int
    n_kv_heads: int
    d_head: int
    rms_eps: float
    qk_norm: bool
    rope_theta: float
    sliding_window: int = 0  # 0 = global attention
    rope_style: int = ROPE_INTERLEAVED

    @property
    def n_kv_cols(self) -> int:
        """Width of the fused [W_K | W_V] projection."""
        return 2 * self.n_kv_heads * self.d_head

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


SMOLLM2_135M = LayerShape("smollm2-135m", 576, 9, 3, 64, 1e-5, False, 1.0e4)
GEMMA3_4B_GLOBAL = LayerShape("gemma3-4b-global", 2560, 8, 4, 256, 1e-6, True, 1.0e6)
GEMMA3_4B_LOCAL = LayerShape("gemma3-4b-local", 2560, 8, 4, 256, 1e-6, True, 1.0e4, sliding_window=1024)
QWEN3_4B = LayerShape("qwen3-4b", 2560, 32, 8, 128, 1e-6, True, 1.0e6)

# scaled-down layer shapes for tests the fp64 oracle must finish quickly
TINY_GQA = LayerShape("tiny-gqa", 128, 4, 2, 64, 1e-6, True, 1.0e4)
TINY_MHA = LayerShape("tiny-mha", 64, 2, 2, 64, 1e-5, False, 1.0e4)


@dataclass
class LayerWeights:
    """bf16 bit patterns of the tensors one layer's K/V recomputation needs."""

    w_kv: np.ndarray  # [d_hidden, 2*n_kv*d_head]; K columns first, then V columns
    gamma_in: np.ndarray  # [d_hidden] effective pre-attention RMSNorm scale
    gamma_k: Optional[np.ndarray]  # [d_head] per-head key-norm scale, or None


def make_layer_weights(shape: LayerShape, layer: int = 0) -> LayerWeights:
    rng_w = np.random.Generator(np.random.PCG64(SEED_WEIGHTS + layer))
    rng_n = np.random.Generator(np.random.PCG64(SEED_NORMS + layer))
    w_kv = _normal_bf16(rng_w, (shape.d_hidden, shape.n_kv_cols), 0.02)
    gamma_in = _normal_bf16(rng_n, (shape.d_hidden,), 0.02, mean=1.0)
    gamma_k = _normal_bf16(rng_n, (shape.d_head,), 0.02, mean=1.0) if shape.qk_norm else None
    return LayerWeights(w_kv, gamma_in, gamma_k)


def outlier_channels(d_hidden: int, fraction: float = 0.01) -> np.ndarray:
    """Indices of the channels that carry outliers (same set for every row)."""
    rng = np.random.Generator(np.random.PCG64(SEED_OUTLIERS))
    k = int(round(fraction * d_hidden))
    return np.sort(rng.choice(d_hidden, size=k, replace=False))


def make_residuals(shape: LayerShape, n_rows: int, seed: int = 0, outliers: bool = False) -> np.ndarray:
    """Residual rows [n_rows, d_hidden] ~ N(0,1), optionally with 1 % channels scaled by 20."""
    rng = np.random.Generator(np.random.PCG64(SEED_RESIDUALS + seed))
    x = rng.standard_normal(size=(n_rows, shape.d_hidden), dtype=np.float32)
    if outliers:
        x[:, outlier_channels(shape.d_hidden)] *= np.float32(20.0)
    return f32_to_bf16_bits(x)


def make_query(shape: LayerShape, batch: int, seed: int = 0) -> np.ndarray:
    """Query rows [batch, n_q, d_head] ~ N(0,1) (already normed and rotated, as the attention call expects)."""
    rng = np.random.Generator(np.random.PCG64(SEED_QUERY + seed))
    return _normal_bf16(rng, (batch, shape.n_q_heads, shape.d_head), 1.0)


def make_kv(shape: LayerShape, n_keys: int, seed: int = 0, std: float = 1.0):
    """Random stored keys and values, each [n_keys, n_kv, d_head]."""
    rng = np.random.Generator(np.random.PCG64(SEED_KV + seed))
    k = _normal_bf16(rng, (n_keys, shape.n_kv_heads, shape.d_head), std)
    v = _normal_bf16(rng, (n_keys, shape.n_kv_heads, shape.d_head), std)
    return k, v


def make_token_ids(n: int, vocab: int, seed: int = 0) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(SEED_TOKENS + seed))
    return rng.integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)


# --------------------------------------------------------------------------- small stacks
@dataclass(frozen=True)
class StackShape:
    """A whole decoder stack: per-layer attention shape plus MLP width and vocabulary."""

    name: str
    n_layers: int
    d_hidden: int
    n_q_heads: int
    n_kv_heads: int
    d_head: int
    d_mlp: int
    vocab: int
    rms_eps: float
    qk_norm: bool
    theta_global: float
    theta_local: float
    sliding_window: int  # window of the local layers; 0 = every layer is global
    global_every: int  # layer l is global iff l % global_every == global_every - 1 (0 = all global)
    activation: str  # "gelu_tanh" or "silu"
    rope_style: int = ROPE_INTERLEAVED

    def is_global(self, layer: int) -> bool:
        if self.sliding_window == 0 or self.global_every == 0:
            return True
        return layer % self.global_every == self.global_every - 1

    def layer_shape(self, layer: int) -> LayerShape:
        glob = self.is_global(layer)
        return LayerShape(
            f"{self.name}-l{layer}",
            self.d_hidden,
            self.n_q_heads,
            self.n_kv_heads,
            self.d_head,
            self.rms_eps,
            self.qk_norm,
            self.theta_global if glob else self.theta_local,
            0 if glob else self.sliding_window,
            self.rope_style,
        )


# one full local/global period of the Gemma pattern, small enough for an fp64 CPU run
S_GEMMA = StackShape("s-gemma", 6, 256, 4, 2, 64, 512, 2048, 1e-6, True, 1.0e6, 1.0e4, 32, 6, "gelu_tanh")
S_QWEN = StackShape("s-qwen", 4, 256, 8, 2, 64, 512, 2048, 1e-6, True, 1.0e6, 1.0e6, 0, 0, "silu")
S_SMOL = StackShape("s-smol", 4, 192, 3, 1, 64, 384, 1024, 1e-5, False, 1.0e4, 1.0e4, 0, 0, "silu")

GEMMA3_4B_STACK = StackShape(
    "gemma3-4b", 34, 2560, 8, 4, 256, 10240, 262144, 1e-6, True, 1.0e6, 1.0e4, 1024, 6, "gelu_tanh"
)
QWEN3_4B_STACK = StackShape("qwen3-4b", 36, 2560, 32, 8, 128, 9728, 151936, 1e-6, True, 1.0e6, 1.0e6, 0, 0, "silu")


@dataclass
class StackWeights:
    """bf16 bit patterns of every tensor of a small stack."""

    embed: np.ndarray  # [vocab, d_hidden]
    lm_head: np.ndarray  # [d_hidden, vocab]  (untied)
    gamma_final: np.ndarray  # [d_hidden]
    layers: List[Dict[str, np.ndarray]]  # per layer: w_q, w_kv, w_o, w_gate, w_up, w_down, gamma_in, gamma_mlp, gamma_q, gamma_k


def make_stack_weights(stack: StackShape, seed: int = 0) -> StackWeights:
    base = 100 * seed
    rng_e = np.random.Generator(np.random.PCG64(SEED_WEIGHTS + 900 + base))
    # embeddings ~N(0,1) so that residual rows have unit scale; everything else N(0, 0.02)
    embed = _normal_bf16(rng_e, (stack.vocab, stack.d_hidden), 1.0)
    lm_head = _normal_bf16(rng_e, (stack.d_hidden, stack.vocab), 0.02)
    gamma_final = _normal_bf16(rng_e, (stack.d_hidden,), 0.02, mean=1.0)
    layers = []
    nq, nkv, dh, d = stack.n_q_heads, stack.n_kv_heads, stack.d_head, stack.d_hidden
    for l in range(stack.n_layers):
        rw = np.random.Generator(np.random.PCG64(SEED_WEIGHTS + base + l))
        rn = np.random.Generator(np.random.PCG64(SEED_NORMS + base + l))
        lw = {
            "w_kv": _normal_bf16(rw, (d, 2 * nkv * dh), 0.02),
            "w_q": _normal_bf16(rw, (d, nq * dh), 0.02),
            "w_o": _normal_bf16(rw, (nq * dh, d), 0.02),
            "w_gate": _normal_bf16(rw, (d, stack.d_mlp), 0.02),
            "w_up": _normal_bf16(rw, (d, stack.d_mlp), 0.02),
            "w_down": _normal_bf16(rw, (stack.d_mlp, d), 0.02),
            "gamma_in": _normal_bf16(rn, (d,), 0.02, mean=1.0),
            "gamma_mlp": _normal_bf16(rn, (d,), 0.02, mean=1.0),
        }
        if stack.qk_norm:
            lw["gamma_q"] = _normal_bf16(rn, (dh,), 0.02, mean=1.0)
            lw["gamma_k"] = _normal_bf16(rn, (dh,), 0.02, mean=1.0)
        layers.append(lw)
    return StackWeights(embed, lm_head, gamma_final, layers)


def with_style(shape: LayerShape, rope_style: int) -> LayerShape:
    return replace(shape, rope_style=rope_style)
