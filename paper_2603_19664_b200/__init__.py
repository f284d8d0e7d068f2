"""KV-Direct hot path for NVIDIA B200: K/V recomputation from checkpointed residual rows and
decode attention, as hand-written sm_100a kernels behind a C ABI (``include/kvd.h``).

``binding`` is a thin ctypes layer over ``libkvd.so``; ``build`` compiles the library in-tree.
"""
from .binding import (KVD_MAX_SEGMENTS, KVD_OK, KVD_ROPE_HALF, KVD_ROPE_INTERLEAVED, EXPORTED_SYMBOLS, Kvd, KvdError,
                      kvd_attention_split, kvd_fused_recompute_pays, kvd_decode_attention_static, kvd_store_bytes, kvd_store_bytes_dtype, kvd_store_bytes_fp8, kvd_store_bytes_fp4, kvd_fp4_scratch_bytes, kvd_version, kvd_workspace_bytes, load, make_desc,
                      status_string)

__all__ = ["KVD_MAX_SEGMENTS", "KVD_OK", "KVD_ROPE_HALF", "KVD_ROPE_INTERLEAVED", "EXPORTED_SYMBOLS", "Kvd", "KvdError",
           "kvd_attention_split", "kvd_fused_recompute_pays", "kvd_decode_attention_static", "kvd_store_bytes", "kvd_store_bytes_dtype", "kvd_store_bytes_fp8", "kvd_store_bytes_fp4", "kvd_fp4_scratch_bytes", "kvd_version", "kvd_workspace_bytes", "load", "make_desc", "status_string"]
