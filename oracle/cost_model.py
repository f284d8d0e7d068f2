"""Closed forms of the paper's memory and cost model (Eq. 23-28) -- TEST INFRASTRUCTURE ONLY.

Each function is one equation written out.  Pinned by the values the paper prints for its
Gemma-3-4B worked example and by the six rows of its Table 1 (tests/golden/table1_memory.txt).
"""
from __future__ import annotations


def kv_bytes_per_token(n_layers: int, n_kv: int, d_head: int, b: int = 2) -> int:
    """Eq. 23: bytes of K and V one token occupies across all layers."""
    return 2 * n_layers * n_kv * d_head * b


def residual_bytes_per_token(d_hidden: int, b: int = 2) -> int:
    """Eq. 24: bytes of one residual checkpoint."""
    return d_hidden * b


def compression_ratio(n_layers: int, n_kv: int, d_head: int, d_hidden: int) -> float:
    """Eq. 25: rho = 2 L n_kv d_head / d_hidden."""
    return 2.0 * n_layers * n_kv * d_head / d_hidden


def recompute_flops(n_tokens: int, n_kv: int, d_hidden: int, d_head: int) -> int:
    """Eq. 26: flops to rebuild K and V of n_tokens at one layer."""
    return 4 * n_tokens * n_kv * d_hidden * d_head


def read_bytes(n_tokens: int, n_kv: int, d_head: int, b: int = 2) -> int:
    """Eq. 27: bytes moved when the same K and V are read from a cache at one layer."""
    return 2 * n_tokens * n_kv * d_head * b


def total_memory(T: int, B: int, n_layers: int, n_kv: int, d_head: int, d_hidden: int, b: int = 2) -> int:
    """Eq. 28: B live K/V entries per layer plus T-B residual checkpoints (one vector per token)."""
    return 2 * B * n_layers * n_kv * d_head * b + (T - B) * d_hidden * b


def per_layer_checkpoint_memory(T: int, B: int, n_layers: int, n_kv: int, d_head: int, d_hidden: int,
                                b: int = 2) -> int:
    """Memory when the residual entering *every* layer is checkpointed, which is what a per-layer
    recompute (Algorithm 1's STORE_RESIDUAL(C, l) inside the layer loop) needs: Eq. 28 with the
    second term multiplied by L."""
    return 2 * B * n_layers * n_kv * d_head * b + (T - B) * n_layers * d_hidden * b
