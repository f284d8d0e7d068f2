"""ctypes binding of ``libkvd.so`` -- argument marshalling only.

Every function here has the name of the C entry point it calls (``include/kvd.h``) and does nothing
but convert Python / torch objects to pointers and sizes.  K/V recomputation and attention run
entirely inside the CUDA kernels of the library; there is no Python or CPU fallback: if the library
is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
# KVD_LIBRARY=check selects the checking build (libkvd_check.so: device-side index tests, see kvd.h); a path selects
# that file.  Either way it is this library's own code: there is no other implementation to fall back to.
_sel = os.environ.get("KVD_LIBRARY", "")
LIB_PATH = (os.path.join(_HERE, "libkvd_check.so") if _sel == "check" else _sel) if _sel else os.path.join(_HERE, "libkvd.so")

KVD_OK = 0
KVD_ERR_INVALID_ARG = 1
KVD_ERR_SHAPE = 2
KVD_ERR_ALIGNMENT = 3
KVD_ERR_CAPACITY = 4
KVD_ERR_STATE = 5
KVD_ERR_UNSUPPORTED = 6
KVD_ERR_CUDA = 7
KVD_ERR_TIMEOUT = 8
KVD_ERR_POSITION = 9
KVD_ERR_BOUNDS = 10
KVD_ROPE_INTERLEAVED = 0
KVD_ROPE_HALF = 1
KVD_MAX_SEGMENTS = 4

# every symbol include/kvd.h declares
EXPORTED_SYMBOLS = (
    "kvd_create", "kvd_destroy", "kvd_set_layer", "kvd_store_bytes", "kvd_attach_store", "kvd_reset_sequence",
    "kvd_decode_attention_recompute", "kvd_fused_recompute_pays", "kvd_decode_attention_recompute_fp8", "kvd_set_dtype", "kvd_store_bytes_dtype",
    "kvd_quantize_rows_fp8", "kvd_recompute_kv_fp8_rows", "kvd_decode_attention_recompute_fp8_rows",
    "kvd_store_bytes_fp8", "kvd_attach_store_fp8", "kvd_rows_stored_fp8", "kvd_reset_sequence_fp8", "kvd_checkpoint_residual_fp8", "kvd_recompute_kv_fp8",
    "kvd_store_bytes_fp4", "kvd_attach_store_fp4", "kvd_rows_stored_fp4", "kvd_reset_sequence_fp4",
    "kvd_checkpoint_residual_fp4", "kvd_fp4_scratch_bytes", "kvd_recompute_kv_fp4",
    "kvd_rows_stored", "kvd_workspace_bytes", "kvd_attention_split", "kvd_attach_workspace", "kvd_checkpoint_residual", "kvd_checkpoint_residual_step", "kvd_decode_step_kv", "kvd_recompute_kv",
    "kvd_recompute_kv_step",
    "kvd_decode_attention", "kvd_decode_attention_rows", "kvd_prefill_attention", "kvd_decode_attention_static", "kvd_memory_stats", "kvd_poll_status", "kvd_selftest_wait_timeout", "kvd_build_has_checks", "kvd_selftest_bounds_check", "kvd_set_trace", "kvd_launch_count", "kvd_last_cuda_error",
    "kvd_status_string", "kvd_version",
    # include/kvd_scaffold.h: the parts of a decoder layer around the hot path, for whole-stack tests and benchmarks
    "kvd_scaffold_linear_create", "kvd_scaffold_linear_destroy", "kvd_scaffold_linear_out_cols", "kvd_scaffold_linear",
    "kvd_scaffold_query_finish", "kvd_scaffold_add_rows", "kvd_scaffold_gated_act", "kvd_scaffold_embed",
    "kvd_scaffold_argmax",
)
KVD_ACT_GELU_TANH = 0
KVD_ACT_SILU = 1


class kvd_store_range(ctypes.Structure):
    _fields_ = [("seq", ctypes.c_int32), ("first_row", ctypes.c_int32), ("n", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("k_out", ctypes.c_void_p), ("v_out", ctypes.c_void_p)]


class kvd_fp8_rows(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("sumsq", ctypes.c_void_p),
                ("positions", ctypes.c_void_p), ("n", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("k_out", ctypes.c_void_p), ("v_out", ctypes.c_void_p)]


class kvd_model_desc(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("d_hidden", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("d_head", ctypes.c_int32), ("rms_eps", ctypes.c_float),
                ("qk_norm", ctypes.c_int32), ("qk_norm_eps", ctypes.c_float), ("rope_style", ctypes.c_int32),
                ("max_seqs", ctypes.c_int32), ("max_tokens_per_seq", ctypes.c_int32), ("max_batch", ctypes.c_int32)]


class kvd_layer_desc(ctypes.Structure):
    _fields_ = [("w_kv", ctypes.c_void_p), ("gamma_in", ctypes.c_void_p), ("gamma_k", ctypes.c_void_p),
                ("rope_theta", ctypes.c_float), ("sliding_window", ctypes.c_int32)]


class kvd_kv_segment(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("row_stride", ctypes.c_int64),
                ("first_pos", ctypes.c_int32), ("len", ctypes.c_int32)]


class kvd_mem_stats(ctypes.Structure):
    _fields_ = [("checkpoint_bytes_used", ctypes.c_uint64), ("checkpoint_bytes_capacity", ctypes.c_uint64),
                ("workspace_bytes", ctypes.c_uint64), ("prepared_weight_bytes", ctypes.c_uint64),
                ("tokens_stored", ctypes.c_uint64), ("eq23_kv_bytes_per_token", ctypes.c_uint64),
                ("eq24_residual_bytes_per_token", ctypes.c_uint64),
                ("per_layer_residual_bytes_per_token", ctypes.c_uint64)]


class KvdError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        self.status = status
        msg = f"{what}: {status_string(status)} (status {status})"
        if detail:
            msg += f" [{detail}]"
        super().__init__(msg)


_lib: Optional[ctypes.CDLL] = None


def load() -> ctypes.CDLL:
    """Load libkvd.so (built by ``paper_2603_19664_b200.build``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2603_19664_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
    lib.kvd_create.argtypes = [ctypes.POINTER(kvd_model_desc), ctypes.POINTER(vp)]
    lib.kvd_create.restype = i32
    lib.kvd_destroy.argtypes = [vp]
    lib.kvd_destroy.restype = None
    lib.kvd_set_layer.argtypes = [vp, i32, ctypes.POINTER(kvd_layer_desc), vp]
    lib.kvd_set_layer.restype = i32
    lib.kvd_store_bytes.argtypes = [ctypes.POINTER(kvd_model_desc), i32]
    lib.kvd_store_bytes.restype = sz
    lib.kvd_store_bytes_dtype.argtypes = [ctypes.POINTER(kvd_model_desc), i32, i32]
    lib.kvd_store_bytes_dtype.restype = sz
    lib.kvd_attach_store.argtypes = [vp, vp, sz, i32]
    lib.kvd_attach_store.restype = i32
    lib.kvd_reset_sequence.argtypes = [vp, i32]
    lib.kvd_reset_sequence.restype = i32
    lib.kvd_rows_stored.argtypes = [vp, i32, i32]
    lib.kvd_rows_stored.restype = i32
    lib.kvd_workspace_bytes.argtypes = [ctypes.POINTER(kvd_model_desc)]
    lib.kvd_workspace_bytes.restype = sz
    lib.kvd_attach_workspace.argtypes = [vp, vp, sz]
    lib.kvd_attach_workspace.restype = i32
    lib.kvd_attention_split.argtypes = [i32, i32, i32, i32, ctypes.POINTER(ctypes.c_int32)]
    lib.kvd_attention_split.restype = i32
    lib.kvd_checkpoint_residual.argtypes = [vp, i32, i32, vp, vp, i32, vp]
    lib.kvd_checkpoint_residual.restype = i32
    lib.kvd_checkpoint_residual_step.argtypes = [vp, i32, i32, ctypes.POINTER(ctypes.c_int32), vp, vp, vp]
    lib.kvd_checkpoint_residual_step.restype = i32
    lib.kvd_recompute_kv.argtypes = [vp, i32, vp, vp, i32, i32, i32, vp, vp, i64, vp]
    lib.kvd_recompute_kv.restype = i32
    lib.kvd_recompute_kv_step.argtypes = [vp, i32, ctypes.POINTER(kvd_store_range), i32, vp, vp, i32, vp, vp, i64, vp]
    lib.kvd_recompute_kv_step.restype = i32
    lib.kvd_decode_step_kv.argtypes = [vp, i32, ctypes.POINTER(kvd_store_range), i32, i64, vp, vp, i32,
                                       ctypes.POINTER(ctypes.c_int32), vp, vp, i64, vp]
    lib.kvd_decode_step_kv.restype = i32
    lib.kvd_decode_attention.argtypes = [vp, i32, i32, vp, ctypes.POINTER(ctypes.c_int32),
                                         ctypes.POINTER(kvd_kv_segment), i32, ctypes.c_float, vp, vp]
    lib.kvd_decode_attention.restype = i32
    lib.kvd_fused_recompute_pays.argtypes = [ctypes.POINTER(kvd_model_desc), i64, i32]
    lib.kvd_fused_recompute_pays.restype = i32
    lib.kvd_store_bytes_fp4.argtypes = [ctypes.POINTER(kvd_model_desc), i32]
    lib.kvd_store_bytes_fp4.restype = sz
    lib.kvd_fp4_scratch_bytes.argtypes = [ctypes.POINTER(kvd_model_desc), i32]
    lib.kvd_fp4_scratch_bytes.restype = sz
    lib.kvd_attach_store_fp4.argtypes = [vp, vp, sz, i32]
    lib.kvd_attach_store_fp4.restype = i32
    lib.kvd_rows_stored_fp4.argtypes = [vp, i32, i32]
    lib.kvd_rows_stored_fp4.restype = i32
    lib.kvd_reset_sequence_fp4.argtypes = [vp, i32]
    lib.kvd_reset_sequence_fp4.restype = i32
    lib.kvd_checkpoint_residual_fp4.argtypes = [vp, i32, i32, vp, vp, i32, vp]
    lib.kvd_checkpoint_residual_fp4.restype = i32
    lib.kvd_recompute_kv_fp4.argtypes = [vp, i32, ctypes.POINTER(kvd_store_range), i32, i64, vp, sz, vp]
    lib.kvd_recompute_kv_fp4.restype = i32
    lib.kvd_decode_attention_rows.argtypes = [vp, i32, i32, vp, ctypes.POINTER(ctypes.c_int32),
                                              ctypes.POINTER(kvd_kv_segment), i32, ctypes.c_float, vp, vp]
    lib.kvd_decode_attention_rows.restype = i32
    lib.kvd_prefill_attention.argtypes = [vp, i32, i32, vp, vp, ctypes.POINTER(kvd_kv_segment), i32, ctypes.c_float, vp, vp]
    lib.kvd_prefill_attention.restype = i32
    lib.kvd_set_dtype.argtypes = [vp, i32]
    lib.kvd_set_dtype.restype = i32
    lib.kvd_store_bytes_fp8.argtypes = [ctypes.POINTER(kvd_model_desc), i32]
    lib.kvd_store_bytes_fp8.restype = sz
    lib.kvd_attach_store_fp8.argtypes = [vp, vp, sz, i32]
    lib.kvd_attach_store_fp8.restype = i32
    lib.kvd_rows_stored_fp8.argtypes = [vp, i32, i32]
    lib.kvd_rows_stored_fp8.restype = i32
    lib.kvd_reset_sequence_fp8.argtypes = [vp, i32]
    lib.kvd_reset_sequence_fp8.restype = i32
    lib.kvd_checkpoint_residual_fp8.argtypes = [vp, i32, i32, vp, vp, i32, vp]
    lib.kvd_checkpoint_residual_fp8.restype = i32
    lib.kvd_recompute_kv_fp8.argtypes = [vp, i32, ctypes.POINTER(kvd_store_range), i32, i64, vp]
    lib.kvd_recompute_kv_fp8.restype = i32
    lib.kvd_decode_attention_recompute.argtypes = [vp, i32, i32, vp, ctypes.POINTER(ctypes.c_int32),
                                                   ctypes.POINTER(kvd_store_range), vp, vp, i32, vp, vp, i64,
                                                   ctypes.POINTER(kvd_kv_segment), i32, ctypes.c_float, vp, vp]
    lib.kvd_decode_attention_recompute.restype = i32
    lib.kvd_decode_attention_recompute_fp8.argtypes = [vp, i32, i32, vp, ctypes.POINTER(ctypes.c_int32),
                                                       ctypes.POINTER(kvd_store_range), ctypes.POINTER(kvd_store_range),
                                                       i32, i64, ctypes.POINTER(kvd_kv_segment), i32, ctypes.c_float,
                                                       vp, vp]
    lib.kvd_decode_attention_recompute_fp8.restype = i32
    lib.kvd_decode_attention_recompute_fp8_rows.argtypes = [vp, i32, i32, vp, ctypes.POINTER(ctypes.c_int32),
                                                            ctypes.POINTER(kvd_store_range), ctypes.POINTER(kvd_store_range),
                                                            i32, ctypes.POINTER(kvd_fp8_rows), i64,
                                                            ctypes.POINTER(kvd_kv_segment), i32, ctypes.c_float, vp, vp]
    lib.kvd_decode_attention_recompute_fp8_rows.restype = i32
    lib.kvd_quantize_rows_fp8.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    lib.kvd_quantize_rows_fp8.restype = i32
    lib.kvd_recompute_kv_fp8_rows.argtypes = [vp, i32, ctypes.POINTER(kvd_store_range), i32, ctypes.POINTER(kvd_fp8_rows),
                                              i64, vp]
    lib.kvd_recompute_kv_fp8_rows.restype = i32
    lib.kvd_decode_attention_static.argtypes = [i32, i32, i32, i32, i32, vp, ctypes.POINTER(ctypes.c_int32),
                                                ctypes.POINTER(kvd_kv_segment), i32, ctypes.c_float, vp, vp]
    lib.kvd_decode_attention_static.restype = i32
    lib.kvd_memory_stats.argtypes = [vp, ctypes.POINTER(kvd_mem_stats)]
    lib.kvd_memory_stats.restype = i32
    lib.kvd_poll_status.argtypes = [vp, vp]
    lib.kvd_poll_status.restype = i32
    lib.kvd_selftest_wait_timeout.argtypes = [vp, i32, vp]
    lib.kvd_selftest_wait_timeout.restype = i32
    lib.kvd_build_has_checks.argtypes = []
    lib.kvd_build_has_checks.restype = i32
    lib.kvd_selftest_bounds_check.argtypes = [vp, vp]
    lib.kvd_selftest_bounds_check.restype = i32
    lib.kvd_set_trace.argtypes = [vp, vp, sz]
    lib.kvd_set_trace.restype = i32
    lib.kvd_launch_count.argtypes = [vp]
    lib.kvd_launch_count.restype = ctypes.c_uint64
    lib.kvd_last_cuda_error.argtypes = [vp]
    lib.kvd_last_cuda_error.restype = ctypes.c_char_p
    lib.kvd_status_string.argtypes = [i32]
    lib.kvd_status_string.restype = ctypes.c_char_p
    lib.kvd_version.argtypes = []
    lib.kvd_version.restype = ctypes.c_char_p
    lib.kvd_scaffold_linear_create.argtypes = [vp, vp, vp, i32, i32, ctypes.c_float, vp, ctypes.POINTER(vp)]
    lib.kvd_scaffold_linear_create.restype = i32
    lib.kvd_scaffold_linear_destroy.argtypes = [vp, vp]
    lib.kvd_scaffold_linear_destroy.restype = None
    lib.kvd_scaffold_linear_out_cols.argtypes = [vp]
    lib.kvd_scaffold_linear_out_cols.restype = i32
    lib.kvd_scaffold_linear.argtypes = [vp, vp, vp, i32, vp, i64, vp]
    lib.kvd_scaffold_linear.restype = i32
    lib.kvd_scaffold_query_finish.argtypes = [vp, i32, vp, i64, vp, i32, vp, vp, vp]
    lib.kvd_scaffold_query_finish.restype = i32
    lib.kvd_scaffold_add_rows.argtypes = [vp, vp, vp, i64, i32, i32, vp]
    lib.kvd_scaffold_add_rows.restype = i32
    lib.kvd_scaffold_gated_act.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp]
    lib.kvd_scaffold_gated_act.restype = i32
    lib.kvd_scaffold_embed.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp]
    lib.kvd_scaffold_embed.restype = i32
    lib.kvd_scaffold_argmax.argtypes = [vp, vp, i64, i32, i32, vp, vp]
    lib.kvd_scaffold_argmax.restype = i32
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().kvd_status_string(int(status)).decode()


def kvd_version() -> str:
    return load().kvd_version().decode()


def kvd_build_has_checks() -> bool:
    return bool(load().kvd_build_has_checks())


def make_desc(n_layers: int, d_hidden: int, n_q_heads: int, n_kv_heads: int, d_head: int, rms_eps: float,
              qk_norm: bool, qk_norm_eps: float, rope_style: int = KVD_ROPE_INTERLEAVED, max_seqs: int = 1,
              max_tokens_per_seq: int = 4096, max_batch: int = 1) -> kvd_model_desc:
    return kvd_model_desc(n_layers, d_hidden, n_q_heads, n_kv_heads, d_head, rms_eps, 1 if qk_norm else 0,
                          qk_norm_eps, rope_style, max_seqs, max_tokens_per_seq, max_batch)


def kvd_store_bytes(desc: kvd_model_desc, layers_stored: int) -> int:
    return int(load().kvd_store_bytes(ctypes.byref(desc), layers_stored))


def kvd_store_bytes_dtype(desc: kvd_model_desc, layers_stored: int, dtype: int) -> int:
    return int(load().kvd_store_bytes_dtype(ctypes.byref(desc), layers_stored, dtype))


def kvd_store_bytes_fp8(desc: kvd_model_desc, layers_stored: int) -> int:
    return int(load().kvd_store_bytes_fp8(ctypes.byref(desc), layers_stored))


def kvd_store_bytes_fp4(desc: kvd_model_desc, layers_stored: int) -> int:
    return int(load().kvd_store_bytes_fp4(ctypes.byref(desc), layers_stored))


def kvd_fp4_scratch_bytes(desc: kvd_model_desc, max_rows: int) -> int:
    return int(load().kvd_fp4_scratch_bytes(ctypes.byref(desc), max_rows))


def kvd_workspace_bytes(desc: kvd_model_desc) -> int:
    return int(load().kvd_workspace_bytes(ctypes.byref(desc)))


def kvd_fused_recompute_pays(desc: kvd_model_desc, total_rows: int, fp8: bool = False) -> bool:
    return bool(load().kvd_fused_recompute_pays(ctypes.byref(desc), int(total_rows), 1 if fp8 else 0))


def kvd_attention_split(d_head: int, n_kv_heads: int, first_visible: int, last_visible: int) -> Tuple[int, int]:
    """(number of chunks, keys per chunk) of one sequence's visible range; (0, 0) on bad arguments."""
    ck = ctypes.c_int32(0)
    n = int(load().kvd_attention_split(d_head, n_kv_heads, first_visible, last_visible, ctypes.byref(ck)))
    return n, int(ck.value)


def _ptr(t) -> int:
    """Device (or host) address of a torch tensor, or None."""
    return None if t is None else int(t.data_ptr())


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    return int(stream)


Segment = Tuple[object, object, int, int, int]  # (k tensor/ptr, v tensor/ptr, row_stride, first_pos, len)

KVD_STATIC_SCRATCH_BYTES = 8 << 20


def _marshal_segments(batch: int, q_pos, segs):
    n_segs = max((len(s) for s in segs), default=0)
    pos_arr = (ctypes.c_int32 * max(batch, 1))(*[int(p) for p in q_pos])
    seg_arr = (kvd_kv_segment * max(batch * n_segs, 1))()
    for b in range(batch):
        for s in range(n_segs):
            e = seg_arr[b * n_segs + s]
            if s < len(segs[b]):
                k, v, stride, first, ln = segs[b][s]
                e.k = k if isinstance(k, int) else _ptr(k)
                e.v = v if isinstance(v, int) else _ptr(v)
                e.row_stride, e.first_pos, e.len = int(stride), int(first), int(ln)
            else:
                e.k, e.v, e.row_stride, e.first_pos, e.len = None, None, 0, 0, 0
    return n_segs, pos_arr, seg_arr


def kvd_decode_attention_static(n_q_heads: int, n_kv_heads: int, d_head: int, sliding_window: int, batch: int, q,
                                q_pos: Sequence[int], segs: Sequence[Sequence[Segment]], scale: float, out,
                                stream=None) -> int:
    """Decode attention without a context or workspace, for callers that may not allocate device
    memory: the scratch is a fixed array inside the library.  Returns the kvd_status (0 = ok) instead
    of raising, so that a caller can test the capacity limit."""
    n_segs, pos_arr, seg_arr = _marshal_segments(batch, q_pos, segs)
    return int(load().kvd_decode_attention_static(n_q_heads, n_kv_heads, d_head, sliding_window, batch, _ptr(q),
                                                  pos_arr, seg_arr, n_segs, float(scale), _ptr(out),
                                                  _stream(stream)))


class Kvd:
    """One library context.  Method names mirror the C entry points."""

    def __init__(self, desc: kvd_model_desc):
        self._lib = load()
        self.desc = desc
        h = ctypes.c_void_p()
        st = self._lib.kvd_create(ctypes.byref(desc), ctypes.byref(h))
        if st != KVD_OK:
            raise KvdError(st, "kvd_create")
        self._h = h
        self._keep: List[object] = []  # tensors the context borrows (store arena, workspace)

    def close(self) -> None:
        if getattr(self, "_h", None):
            self._lib.kvd_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int, what: str) -> None:
        if st != KVD_OK:
            raise KvdError(st, what, self._lib.kvd_last_cuda_error(self._h).decode())

    def kvd_set_layer(self, layer: int, w_kv, gamma_in, gamma_k, rope_theta: float, sliding_window: int = 0,
                      stream=None) -> None:
        ld = kvd_layer_desc(_ptr(w_kv), _ptr(gamma_in), _ptr(gamma_k), rope_theta, sliding_window)
        self._check(self._lib.kvd_set_layer(self._h, layer, ctypes.byref(ld), _stream(stream)), "kvd_set_layer")

    def kvd_attach_store(self, arena, layers_stored: int) -> None:
        self._keep.append(arena)
        self._check(self._lib.kvd_attach_store(self._h, _ptr(arena), arena.numel() * arena.element_size(),
                                               layers_stored), "kvd_attach_store")

    def kvd_attach_workspace(self, ws) -> None:
        self._keep.append(ws)
        self._check(self._lib.kvd_attach_workspace(self._h, _ptr(ws), ws.numel() * ws.element_size()),
                    "kvd_attach_workspace")

    def kvd_reset_sequence(self, seq: int) -> None:
        self._check(self._lib.kvd_reset_sequence(self._h, seq), "kvd_reset_sequence")

    def kvd_rows_stored(self, layer: int, seq: int) -> int:
        return int(self._lib.kvd_rows_stored(self._h, layer, seq))

    def kvd_checkpoint_residual(self, seq: int, layer: int, rows, positions, n: int, stream=None) -> None:
        self._check(self._lib.kvd_checkpoint_residual(self._h, seq, layer, _ptr(rows), _ptr(positions), n,
                                                      _stream(stream)), "kvd_checkpoint_residual")

    def kvd_checkpoint_residual_step(self, layer: int, seqs: Sequence[int], rows, positions, stream=None) -> None:
        arr = (ctypes.c_int32 * max(len(seqs), 1))(*[int(s) for s in seqs])
        self._check(self._lib.kvd_checkpoint_residual_step(self._h, layer, len(seqs), arr, _ptr(rows), _ptr(positions),
                                                           _stream(stream)), "kvd_checkpoint_residual_step")

    def kvd_recompute_kv(self, layer: int, rows, positions, n: int, k_out, v_out, out_row_stride: int, seq: int = 0,
                         first_row: int = 0, stream=None) -> None:
        self._check(self._lib.kvd_recompute_kv(self._h, layer, _ptr(rows), _ptr(positions), n, seq, first_row,
                                               _ptr(k_out), _ptr(v_out), out_row_stride, _stream(stream)),
                    "kvd_recompute_kv")

    def kvd_recompute_kv_step(self, layer: int, ranges: Sequence[Tuple[int, int, int, object, object]], rows,
                              positions, n_rows: int, k_rows_out, v_rows_out, out_row_stride: int, stream=None) -> None:
        """ranges: (seq, first_row, n, k_out, v_out) per sequence; rows/positions: the new tokens (or None, 0)."""
        arr = (kvd_store_range * max(len(ranges), 1))()
        for i, (seq, first_row, n, k_out, v_out) in enumerate(ranges):
            arr[i].seq, arr[i].first_row, arr[i].n, arr[i].reserved = int(seq), int(first_row), int(n), 0
            arr[i].k_out, arr[i].v_out = _ptr(k_out), _ptr(v_out)
        self._check(self._lib.kvd_recompute_kv_step(self._h, layer, arr, len(ranges), _ptr(rows), _ptr(positions),
                                                    n_rows, _ptr(k_rows_out), _ptr(v_rows_out), out_row_stride,
                                                    _stream(stream)), "kvd_recompute_kv_step")

    def kvd_decode_step_kv(self, layer: int, ranges: Sequence[Tuple[int, int, int, object, object]], out_row_stride: int,
                           rows, positions, n_rows: int, append_seqs: Optional[Sequence[int]], k_rows_out, v_rows_out,
                           rows_out_row_stride: int, stream=None) -> None:
        """ranges as for kvd_recompute_kv_step; append_seqs: the sequence slot each new row is appended to, or None."""
        arr = (kvd_store_range * max(len(ranges), 1))()
        for i, (seq, first_row, n, k_out, v_out) in enumerate(ranges):
            arr[i].seq, arr[i].first_row, arr[i].n, arr[i].reserved = int(seq), int(first_row), int(n), 0
            arr[i].k_out, arr[i].v_out = _ptr(k_out), _ptr(v_out)
        seqs = None if append_seqs is None else (ctypes.c_int32 * max(len(append_seqs), 1))(*[int(x) for x in append_seqs])
        self._check(self._lib.kvd_decode_step_kv(self._h, layer, arr, len(ranges), out_row_stride, _ptr(rows),
                                                 _ptr(positions), n_rows, seqs, _ptr(k_rows_out), _ptr(v_rows_out),
                                                 rows_out_row_stride, _stream(stream)), "kvd_decode_step_kv")

    def kvd_decode_attention(self, layer: int, batch: int, q, q_pos: Sequence[int],
                             segs: Sequence[Sequence[Segment]], scale: float, out, stream=None) -> None:
        n_segs = max((len(s) for s in segs), default=0)
        pos_arr = (ctypes.c_int32 * max(batch, 1))(*[int(p) for p in q_pos])
        seg_arr = (kvd_kv_segment * max(batch * n_segs, 1))()
        for b in range(batch):
            for s in range(n_segs):
                e = seg_arr[b * n_segs + s]
                if s < len(segs[b]):
                    k, v, stride, first, ln = segs[b][s]
                    e.k = k if isinstance(k, int) else _ptr(k)
                    e.v = v if isinstance(v, int) else _ptr(v)
                    e.row_stride, e.first_pos, e.len = int(stride), int(first), int(ln)
                else:
                    e.k, e.v, e.row_stride, e.first_pos, e.len = None, None, 0, 0, 0
        self._check(self._lib.kvd_decode_attention(self._h, layer, batch, _ptr(q), pos_arr, seg_arr, n_segs,
                                                   float(scale), _ptr(out), _stream(stream)), "kvd_decode_attention")

    def kvd_decode_attention_rows(self, layer: int, n_rows: int, q, q_pos: Sequence[int], segs: Sequence[Segment],
                                  scale: float, out, stream=None) -> None:
        """Several query rows of one sequence (segs: that sequence's segments), each with its own position."""
        n_segs, _, seg_arr = _marshal_segments(1, [0], [list(segs)])
        pos_arr = (ctypes.c_int32 * max(n_rows, 1))(*[int(p) for p in q_pos])
        self._check(self._lib.kvd_decode_attention_rows(self._h, layer, n_rows, _ptr(q), pos_arr, seg_arr, n_segs,
                                                        float(scale), _ptr(out), _stream(stream)),
                    "kvd_decode_attention_rows")

    def kvd_prefill_attention(self, layer: int, n_rows: int, q, q_pos_dev, segs: Sequence[Segment], scale: float, out,
                              stream=None) -> None:
        """Many query rows of one sequence in one launch; q_pos_dev: int32 device tensor [n_rows]."""
        n_segs, _, seg_arr = _marshal_segments(1, [0], [list(segs)])
        self._check(self._lib.kvd_prefill_attention(self._h, layer, n_rows, _ptr(q), _ptr(q_pos_dev), seg_arr, n_segs,
                                                    float(scale), _ptr(out), _stream(stream)), "kvd_prefill_attention")

    def kvd_decode_attention_recompute(self, layer: int, batch: int, q, q_pos: Sequence[int],
                                       ranges: Sequence[Tuple[int, int, int]], rows, positions, n_rows: int,
                                       k_rows_out, v_rows_out, out_row_stride: int,
                                       segs: Sequence[Sequence[Segment]], scale: float, out, stream=None) -> None:
        """ranges: (seq, first_row, n) per sequence -- attended inside the recompute kernel; rows/positions:
        the new tokens (their K/V are written); segs: the live segments, as for kvd_decode_attention."""
        n_segs, pos_arr, seg_arr = _marshal_segments(batch, q_pos, segs)
        arr = (kvd_store_range * max(len(ranges), 1))()
        for i, (seq, first_row, n) in enumerate(ranges):
            arr[i].seq, arr[i].first_row, arr[i].n, arr[i].reserved = int(seq), int(first_row), int(n), 0
            arr[i].k_out, arr[i].v_out = None, None
        self._check(self._lib.kvd_decode_attention_recompute(
            self._h, layer, batch, _ptr(q), pos_arr, arr, _ptr(rows), _ptr(positions), n_rows, _ptr(k_rows_out),
            _ptr(v_rows_out), out_row_stride, seg_arr, n_segs, float(scale), _ptr(out), _stream(stream)),
            "kvd_decode_attention_recompute")

    def kvd_decode_attention_recompute_fp8(self, layer: int, batch: int, q, q_pos: Sequence[int],
                                           ranges: Sequence[Tuple[int, int, int]],
                                           store_ranges: Sequence[Tuple[int, int, int, object, object]],
                                           out_row_stride: int, segs: Sequence[Sequence[Segment]], scale: float, out,
                                           stream=None) -> None:
        """ranges: (seq, first_row, n) of the FP8 store per sequence -- attended inside the recompute kernel;
        store_ranges: (seq, first_row, n, k_out, v_out) of the FP8 store whose K/V are written."""
        n_segs, pos_arr, seg_arr = _marshal_segments(batch, q_pos, segs)
        arr = (kvd_store_range * max(len(ranges), 1))()
        for i, (seq, first_row, n) in enumerate(ranges):
            arr[i].seq, arr[i].first_row, arr[i].n, arr[i].reserved = int(seq), int(first_row), int(n), 0
            arr[i].k_out, arr[i].v_out = None, None
        sarr = (kvd_store_range * max(len(store_ranges), 1))()
        for i, (seq, first_row, n, k_out, v_out) in enumerate(store_ranges):
            sarr[i].seq, sarr[i].first_row, sarr[i].n, sarr[i].reserved = int(seq), int(first_row), int(n), 0
            sarr[i].k_out, sarr[i].v_out = _ptr(k_out), _ptr(v_out)
        self._check(self._lib.kvd_decode_attention_recompute_fp8(
            self._h, layer, batch, _ptr(q), pos_arr, arr, sarr, len(store_ranges), out_row_stride, seg_arr, n_segs,
            float(scale), _ptr(out), _stream(stream)), "kvd_decode_attention_recompute_fp8")

    @staticmethod
    def _fp8_rows(rows):
        """(codes, scales, sumsq, positions, n, k_out, v_out) -> kvd_fp8_rows, or None."""
        if rows is None:
            return None
        codes, scales, sumsq, positions, n, k_out, v_out = rows
        return kvd_fp8_rows(_ptr(codes), _ptr(scales), _ptr(sumsq), _ptr(positions), int(n), 0, _ptr(k_out), _ptr(v_out))

    def kvd_quantize_rows_fp8(self, rows, n: int, codes_out, scales_out, sumsq_out, stream=None) -> None:
        self._check(self._lib.kvd_quantize_rows_fp8(self._h, _ptr(rows), n, _ptr(codes_out), _ptr(scales_out),
                                                    _ptr(sumsq_out), _stream(stream)), "kvd_quantize_rows_fp8")

    def kvd_recompute_kv_fp8_rows(self, layer: int, ranges: Sequence[Tuple[int, int, int, object, object]], rows,
                                  out_row_stride: int, stream=None) -> None:
        """ranges as for kvd_recompute_kv_fp8; rows: (codes, scales, sumsq, positions, n, k_out, v_out) or None."""
        arr = (kvd_store_range * max(len(ranges), 1))()
        for i, (seq, first_row, n, k_out, v_out) in enumerate(ranges):
            arr[i].seq, arr[i].first_row, arr[i].n, arr[i].reserved = int(seq), int(first_row), int(n), 0
            arr[i].k_out, arr[i].v_out = _ptr(k_out), _ptr(v_out)
        r = self._fp8_rows(rows)
        self._check(self._lib.kvd_recompute_kv_fp8_rows(self._h, layer, arr, len(ranges), ctypes.byref(r) if r else None,
                                                        out_row_stride, _stream(stream)), "kvd_recompute_kv_fp8_rows")

    def kvd_decode_attention_recompute_fp8_rows(self, layer: int, batch: int, q, q_pos: Sequence[int],
                                                ranges: Sequence[Tuple[int, int, int]],
                                                store_ranges: Sequence[Tuple[int, int, int, object, object]], rows,
                                                out_row_stride: int, segs: Sequence[Sequence[Segment]], scale: float,
                                                out, stream=None) -> None:
        """As kvd_decode_attention_recompute_fp8, plus caller-held quantised rows (see kvd_recompute_kv_fp8_rows)."""
        n_segs, pos_arr, seg_arr = _marshal_segments(batch, q_pos, segs)
        arr = (kvd_store_range * max(len(ranges), 1))()
        for i, (seq, first_row, n) in enumerate(ranges):
            arr[i].seq, arr[i].first_row, arr[i].n, arr[i].reserved = int(seq), int(first_row), int(n), 0
            arr[i].k_out, arr[i].v_out = None, None
        sarr = (kvd_store_range * max(len(store_ranges), 1))()
        for i, (seq, first_row, n, k_out, v_out) in enumerate(store_ranges):
            sarr[i].seq, sarr[i].first_row, sarr[i].n, sarr[i].reserved = int(seq), int(first_row), int(n), 0
            sarr[i].k_out, sarr[i].v_out = _ptr(k_out), _ptr(v_out)
        r = self._fp8_rows(rows)
        self._check(self._lib.kvd_decode_attention_recompute_fp8_rows(
            self._h, layer, batch, _ptr(q), pos_arr, arr, sarr, len(store_ranges), ctypes.byref(r) if r else None,
            out_row_stride, seg_arr, n_segs, float(scale), _ptr(out), _stream(stream)),
            "kvd_decode_attention_recompute_fp8_rows")

    def kvd_set_dtype(self, dtype: int) -> None:
        """0 = bf16 (default), 1 = fp16 (checkpoint, recompute and kvd_decode_attention), 2 = fp32 (checkpoint and
        recompute); before kvd_set_layer and kvd_attach_store."""
        self._check(self._lib.kvd_set_dtype(self._h, dtype), "kvd_set_dtype")

    def kvd_attach_store_fp8(self, arena, layers_stored: int) -> None:
        self._keep.append(arena)
        self._check(self._lib.kvd_attach_store_fp8(self._h, _ptr(arena), arena.numel() * arena.element_size(),
                                                   layers_stored), "kvd_attach_store_fp8")

    def kvd_reset_sequence_fp8(self, seq: int) -> None:
        self._check(self._lib.kvd_reset_sequence_fp8(self._h, seq), "kvd_reset_sequence_fp8")

    def kvd_rows_stored_fp8(self, layer: int, seq: int) -> int:
        return int(self._lib.kvd_rows_stored_fp8(self._h, layer, seq))

    def kvd_checkpoint_residual_fp8(self, seq: int, layer: int, rows, positions, n: int, stream=None) -> None:
        self._check(self._lib.kvd_checkpoint_residual_fp8(self._h, seq, layer, _ptr(rows), _ptr(positions), n,
                                                          _stream(stream)), "kvd_checkpoint_residual_fp8")

    def kvd_recompute_kv_fp8(self, layer: int, ranges: Sequence[Tuple[int, int, int, object, object]],
                             out_row_stride: int, stream=None) -> None:
        """ranges: (seq, first_row, n, k_out, v_out) over the FP8 store."""
        arr = (kvd_store_range * max(len(ranges), 1))()
        for i, (seq, first_row, n, k_out, v_out) in enumerate(ranges):
            arr[i].seq, arr[i].first_row, arr[i].n, arr[i].reserved = int(seq), int(first_row), int(n), 0
            arr[i].k_out, arr[i].v_out = _ptr(k_out), _ptr(v_out)
        self._check(self._lib.kvd_recompute_kv_fp8(self._h, layer, arr, len(ranges), out_row_stride, _stream(stream)),
                    "kvd_recompute_kv_fp8")

    def kvd_attach_store_fp4(self, arena, layers_stored: int) -> None:
        self._keep.append(arena)
        self._check(self._lib.kvd_attach_store_fp4(self._h, _ptr(arena), arena.numel() * arena.element_size(),
                                                   layers_stored), "kvd_attach_store_fp4")

    def kvd_reset_sequence_fp4(self, seq: int) -> None:
        self._check(self._lib.kvd_reset_sequence_fp4(self._h, seq), "kvd_reset_sequence_fp4")

    def kvd_rows_stored_fp4(self, layer: int, seq: int) -> int:
        return int(self._lib.kvd_rows_stored_fp4(self._h, layer, seq))

    def kvd_checkpoint_residual_fp4(self, seq: int, layer: int, rows, positions, n: int, stream=None) -> None:
        self._check(self._lib.kvd_checkpoint_residual_fp4(self._h, seq, layer, _ptr(rows), _ptr(positions), n,
                                                          _stream(stream)), "kvd_checkpoint_residual_fp4")

    def kvd_recompute_kv_fp4(self, layer: int, ranges: Sequence[Tuple[int, int, int, object, object]],
                             out_row_stride: int, scratch, stream=None) -> None:
        """ranges: (seq, first_row, n, k_out, v_out) over the FP4 store; scratch: a uint8 device tensor."""
        arr = (kvd_store_range * max(len(ranges), 1))()
        for i, (seq, first_row, n, k_out, v_out) in enumerate(ranges):
            arr[i].seq, arr[i].first_row, arr[i].n, arr[i].reserved = int(seq), int(first_row), int(n), 0
            arr[i].k_out, arr[i].v_out = _ptr(k_out), _ptr(v_out)
        self._check(self._lib.kvd_recompute_kv_fp4(self._h, layer, arr, len(ranges), out_row_stride, _ptr(scratch),
                                                   scratch.numel() * scratch.element_size(), _stream(stream)),
                    "kvd_recompute_kv_fp4")

    def kvd_memory_stats(self) -> dict:
        ms = kvd_mem_stats()
        self._check(self._lib.kvd_memory_stats(self._h, ctypes.byref(ms)), "kvd_memory_stats")
        return {name: int(getattr(ms, name)) for name, _ in kvd_mem_stats._fields_}

    def kvd_poll_status(self, stream=None) -> int:
        return int(self._lib.kvd_poll_status(self._h, _stream(stream)))

    def kvd_selftest_wait_timeout(self, limit_ms: int, stream=None) -> None:
        self._check(self._lib.kvd_selftest_wait_timeout(self._h, limit_ms, _stream(stream)),
                    "kvd_selftest_wait_timeout")

    def kvd_selftest_bounds_check(self, stream=None) -> int:
        """Returns the status (KVD_ERR_UNSUPPORTED in the release build) instead of raising."""
        return int(self._lib.kvd_selftest_bounds_check(self._h, _stream(stream)))

    def kvd_set_trace(self, buf) -> None:
        if buf is None:
            self._check(self._lib.kvd_set_trace(self._h, None, 0), "kvd_set_trace")
        else:
            self._keep.append(buf)
            self._check(self._lib.kvd_set_trace(self._h, _ptr(buf), buf.numel() * buf.element_size()), "kvd_set_trace")

    def kvd_launch_count(self) -> int:
        return int(self._lib.kvd_launch_count(self._h))

    # ---- include/kvd_scaffold.h (marshalling only, like everything above)
    def kvd_scaffold_linear_create(self, w, gamma, k: int, n: int, rms_eps: float = 0.0, stream=None) -> "Linear":
        h = ctypes.c_void_p()
        self._check(self._lib.kvd_scaffold_linear_create(self._h, _ptr(w), _ptr(gamma), k, n, float(rms_eps),
                                                         _stream(stream), ctypes.byref(h)), "kvd_scaffold_linear_create")
        return Linear(self, h, k, n, int(self._lib.kvd_scaffold_linear_out_cols(h)))

    def kvd_scaffold_linear(self, lin: "Linear", x, m: int, out, out_row_stride: int, stream=None) -> None:
        self._check(self._lib.kvd_scaffold_linear(self._h, lin._h, _ptr(x), m, _ptr(out), out_row_stride,
                                                  _stream(stream)), "kvd_scaffold_linear")

    def kvd_scaffold_query_finish(self, layer: int, q_in, in_row_stride: int, positions, m: int, gamma_q, q_out,
                                  stream=None) -> None:
        self._check(self._lib.kvd_scaffold_query_finish(self._h, layer, _ptr(q_in), in_row_stride, _ptr(positions), m,
                                                        _ptr(gamma_q), _ptr(q_out), _stream(stream)),
                    "kvd_scaffold_query_finish")

    def kvd_scaffold_add_rows(self, h, y, y_row_stride: int, m: int, d: int, stream=None) -> None:
        self._check(self._lib.kvd_scaffold_add_rows(self._h, _ptr(h), _ptr(y), y_row_stride, m, d, _stream(stream)),
                    "kvd_scaffold_add_rows")

    def kvd_scaffold_gated_act(self, gate_up, row_stride: int, m: int, width: int, activation: int, out,
                               stream=None) -> None:
        self._check(self._lib.kvd_scaffold_gated_act(self._h, _ptr(gate_up), row_stride, m, width, activation,
                                                     _ptr(out), _stream(stream)), "kvd_scaffold_gated_act")

    def kvd_scaffold_embed(self, table, tokens, m: int, d: int, vocab: int, out, stream=None) -> None:
        self._check(self._lib.kvd_scaffold_embed(self._h, _ptr(table), _ptr(tokens), m, d, vocab, _ptr(out),
                                                 _stream(stream)), "kvd_scaffold_embed")

    def kvd_scaffold_argmax(self, logits, row_stride: int, m: int, n: int, tokens_out, stream=None) -> None:
        self._check(self._lib.kvd_scaffold_argmax(self._h, _ptr(logits), row_stride, m, n, _ptr(tokens_out),
                                                  _stream(stream)), "kvd_scaffold_argmax")


class Linear:
    """Handle of one prepared weight matrix (kvd_scaffold_linear_create); freed with its context or by close()."""

    def __init__(self, ctx: Kvd, h, k: int, n: int, out_cols: int):
        self._ctx, self._h, self.k, self.n, self.out_cols = ctx, h, k, n, out_cols

    def close(self) -> None:
        if self._h and getattr(self._ctx, "_h", None):
            self._ctx._lib.kvd_scaffold_linear_destroy(self._ctx._h, self._h)
        self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
