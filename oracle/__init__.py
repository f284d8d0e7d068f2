"""CPU oracle for the KV-Direct hot path -- TEST INFRASTRUCTURE ONLY.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import this package.
It shares no code with the CUDA path.  The arithmetic lives in ``kvd_oracle.c`` (plain C, fp64,
loops in the order the paper's equations state); this file compiles it with gcc on first use and
wraps it with ctypes.  ``stack.py`` restates the paper's Algorithm 1 on small decoder stacks and
``cost_model.py`` holds the closed forms of Eq. 23-28.

Parity pins for every function are in ``tests/test_oracle_*.py``; nothing here is unpinned.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvd_oracle.c")
_LIB = os.path.join(_HERE, "libkvd_oracle.so")
_lock = threading.Lock()
_lib: Optional[ctypes.CDLL] = None

ROPE_INTERLEAVED = 0
ROPE_HALF = 1


def build(force: bool = False) -> str:
    """Compile kvd_oracle.c into libkvd_oracle.so next to it (no-op if up to date)."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O3", "-march=native", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared",
                   "-fPIC", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        lib.kvd_oracle_rmsnorm.argtypes = [dp, dp, ctypes.c_int, ctypes.c_double, dp]
        lib.kvd_oracle_rmsnorm.restype = None
        lib.kvd_oracle_rope.argtypes = [dp, ctypes.c_int, ctypes.c_int64, ctypes.c_double, ctypes.c_int]
        lib.kvd_oracle_rope.restype = None
        lib.kvd_oracle_recompute_kv.argtypes = [dp, ip, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, dp,
                                                ctypes.c_double, dp, dp, ctypes.c_double, ctypes.c_double,
                                                ctypes.c_int, dp, dp]
        lib.kvd_oracle_recompute_kv.restype = None
        lib.kvd_oracle_decode_attention.argtypes = [dp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int32, dp,
                                                    dp, ip, ctypes.c_int, ctypes.c_double, ctypes.c_int, dp]
        lib.kvd_oracle_decode_attention.restype = ctypes.c_int
        lib.kvd_oracle_max_threads.restype = ctypes.c_int
        lib.kvd_oracle_set_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def _dp(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _ip(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def max_threads() -> int:
    return int(_load().kvd_oracle_max_threads())


def set_threads(n: int) -> None:
    _load().kvd_oracle_set_threads(int(n))


def rmsnorm(x, gamma, eps: float = 0.0) -> np.ndarray:
    """Eq. 1-2 on one vector (eps inside the root; eps=0 is the paper's literal form)."""
    x = _f64(x)
    gamma = _f64(gamma)
    assert x.ndim == 1 and gamma.shape == x.shape
    out = np.empty_like(x)
    _load().kvd_oracle_rmsnorm(_dp(x), _dp(gamma), x.shape[0], float(eps), _dp(out))
    return out


def rope(x, pos: int, theta: float, style: int = ROPE_INTERLEAVED) -> np.ndarray:
    """Eq. 11-12 on one d_head vector; returns a rotated copy."""
    out = _f64(x).copy()
    assert out.ndim == 1 and out.shape[0] % 2 == 0
    _load().kvd_oracle_rope(_dp(out), out.shape[0], int(pos), float(theta), int(style))
    return out


def recompute_kv(X, pos, gamma_in, W_kv, n_kv: int, d_head: int, rms_eps: float, theta: float,
                 gamma_k=None, qk_eps: float = 0.0, rope_style: int = ROPE_INTERLEAVED) -> Tuple[np.ndarray, np.ndarray]:
    """O1 -- Eq. 13-14: (K, V), each [n, n_kv, d_head] in fp64, from residual rows X [n, d_hidden]."""
    X = _f64(X)
    n, d_hidden = X.shape
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    assert pos.shape == (n,)
    gamma_in = _f64(gamma_in)
    W_kv = _f64(W_kv)
    assert gamma_in.shape == (d_hidden,)
    assert W_kv.shape == (d_hidden, 2 * n_kv * d_head)
    gk = None
    if gamma_k is not None:
        gk = _f64(gamma_k)
        assert gk.shape == (d_head,)
    K = np.empty((n, n_kv, d_head), dtype=np.float64)
    V = np.empty((n, n_kv, d_head), dtype=np.float64)
    _load().kvd_oracle_recompute_kv(_dp(X), _ip(pos), n, d_hidden, n_kv, d_head, _dp(gamma_in), float(rms_eps),
                                    _dp(W_kv), _dp(gk) if gk is not None else None, float(qk_eps), float(theta),
                                    int(rope_style), _dp(K), _dp(V))
    return K, V


def decode_attention(q, q_pos: int, segments: Sequence[Tuple[np.ndarray, np.ndarray, int]], scale: float,
                     window: int = 0) -> np.ndarray:
    """O2 -- Eq. 6-7 for one sequence.

    ``q`` is [n_q, d_head]; ``segments`` is a list of (K, V, first_pos) with K, V [len, n_kv, d_head]
    holding the keys at positions first_pos .. first_pos+len-1 (the recomputed keys, the live window
    and the current token, in Algorithm 1's CONCAT order).  Returns [n_q, d_head] in fp64.
    """
    q = _f64(q)
    n_q, d_head = q.shape
    ks, vs, ps = [], [], []
    n_kv = None
    for (K, V, first) in segments:
        K = _f64(K)
        V = _f64(V)
        assert K.shape == V.shape and K.ndim == 3 and K.shape[2] == d_head
        n_kv = K.shape[1] if n_kv is None else n_kv
        assert K.shape[1] == n_kv
        ks.append(K)
        vs.append(V)
        ps.append(np.arange(first, first + K.shape[0], dtype=np.int32))
    assert n_kv is not None, "at least one segment is required"
    Kc = np.ascontiguousarray(np.concatenate(ks, axis=0))
    Vc = np.ascontiguousarray(np.concatenate(vs, axis=0))
    pc = np.ascontiguousarray(np.concatenate(ps, axis=0))
    out = np.zeros((n_q, d_head), dtype=np.float64)
    _load().kvd_oracle_decode_attention(_dp(q), n_q, n_kv, d_head, int(q_pos), _dp(Kc), _dp(Vc), _ip(pc),
                                        Kc.shape[0], float(scale), int(window), _dp(out))
    return out
