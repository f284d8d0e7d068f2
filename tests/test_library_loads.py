"""CPU-only checks of the C-ABI library: it builds, loads without a GPU driver and exports every
symbol include/kvd.h declares; host-side argument checks that need no device."""
import ctypes
import os
import re

import paper_2603_19664_b200 as kvd
from paper_2603_19664_b200 import binding
from paper_2603_19664_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build()
    lib = ctypes.CDLL(path)
    declared = set()
    for name in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if name.endswith(".h"):
            declared |= set(re.findall(r"\b(kvd_[a-z_0-9]+)\s*\(", open(os.path.join(ROOT, "include", name)).read()))
    declared -= {"kvd_ctx", "kvd_fp8_rows"}
    assert declared == set(binding.EXPORTED_SYMBOLS)
    for name in sorted(declared):
        assert hasattr(lib, name), name


def test_version_and_status_strings():
    assert kvd.kvd_version() == "0.1"
    assert kvd.status_string(0) == "ok"
    for s in range(1, 11):
        assert kvd.status_string(s) not in ("ok", "unknown status")


def test_size_queries_validate_shapes_without_a_device():
    good = kvd.make_desc(34, 2560, 8, 4, 256, 1e-6, True, 1e-6, max_seqs=2, max_tokens_per_seq=4096, max_batch=2)
    # rows + positions for 1 layer: 2 seqs * 4096 tokens * (2560 * 2 + 4) bytes
    assert kvd.kvd_store_bytes(good, 1) == 2 * 4096 * (2560 * 2 + 4 + 4)
    assert kvd.kvd_store_bytes_dtype(good, 1, 1) == kvd.kvd_store_bytes(good, 1)      # fp16: the same room
    assert kvd.kvd_store_bytes_dtype(good, 1, 2) == 2 * 4096 * (2560 * 4 + 4 + 4)     # fp32 rows
    assert kvd.kvd_store_bytes_dtype(good, 1, 3) == 0
    assert kvd.kvd_workspace_bytes(good) > 0
    bad_head = kvd.make_desc(1, 2560, 8, 4, 96, 1e-6, True, 1e-6)
    assert kvd.kvd_store_bytes(bad_head, 1) == 0
    bad_hidden = kvd.make_desc(1, 2500, 8, 4, 256, 1e-6, True, 1e-6)
    assert kvd.kvd_workspace_bytes(bad_hidden) == 0
    bad_group = kvd.make_desc(1, 2560, 7, 4, 256, 1e-6, True, 1e-6)
    assert kvd.kvd_workspace_bytes(bad_group) == 0


def test_create_rejects_bad_arguments_before_touching_a_device():
    lib = binding.load()
    h = ctypes.c_void_p()
    assert lib.kvd_create(None, ctypes.byref(h)) == binding.KVD_ERR_INVALID_ARG
    bad = kvd.make_desc(1, 2560, 8, 4, 96, 1e-6, True, 1e-6)
    assert lib.kvd_create(ctypes.byref(bad), ctypes.byref(h)) == binding.KVD_ERR_SHAPE
    assert not h.value
    # NULL contexts are rejected, not dereferenced
    assert lib.kvd_poll_status(None, None) == binding.KVD_ERR_INVALID_ARG
    assert lib.kvd_rows_stored(None, 0, 0) == -1
    assert lib.kvd_launch_count(None) == 0


def test_attention_split_is_a_function_of_the_visible_range_only():
    """Host logic of the split decode attention uses: bounded chunk counts, chunks of at least two
    iterations aligned to absolute position, full coverage, one wave of CTAs for a long single
    sequence; bad arguments give 0."""
    assert kvd.kvd_attention_split(96, 4, 0, 10) == (0, 0)
    assert kvd.kvd_attention_split(256, 0, 0, 10)[0] == 0
    assert kvd.kvd_attention_split(256, 4, 5, 4)[0] == 0
    assert kvd.kvd_attention_split(256, 4, -1, 4)[0] == 0
    for d_head, n_kv, per_iter in ((256, 4, 32), (128, 8, 64), (64, 3, 128)):
        for span in (1, 2, 31, 33, 257, 1024, 1025, 2049, 4097, 8192, 8193, 32769, 131073, 1000003):
            for lo in (0, 7, 1000, 123457):
                hi = lo + span - 1
                n, ck = kvd.kvd_attention_split(d_head, n_kv, lo, hi)
                assert ck % per_iter == 0 and ck >= 2 * per_iter   # whole iterations, at least two
                assert ck <= 64 * per_iter                                # iteration count is capped
                assert (lo // ck + n - 1) * ck <= hi < (lo // ck + n) * ck  # the chunks cover [lo, hi]
                if span <= 8192:
                    assert n <= 130
                elif ck < 64 * per_iter:
                    assert n <= 592 // n_kv + 2
                # the same visible range in any segment layout or batch gives the same split: it is a pure function
                assert (n, ck) == kvd.kvd_attention_split(d_head, n_kv, lo, hi)
    # a long single sequence of the Gemma-shaped layer: one wave of four CTAs per SM
    n, ck = kvd.kvd_attention_split(256, 4, 0, 32768)
    assert 4 * n <= 4 * 148 and n >= 140 and ck == 224


def test_entry_points_reject_null_contexts_and_bad_shapes_without_a_device():
    lib = binding.load()
    assert lib.kvd_recompute_kv_step(None, 0, None, 0, None, None, 0, None, None, 0, None) == binding.KVD_ERR_INVALID_ARG
    assert lib.kvd_recompute_kv(None, 0, None, None, 0, 0, 0, None, None, 0, None) == binding.KVD_ERR_INVALID_ARG
    assert lib.kvd_decode_attention(None, 0, 0, None, None, None, 0, 0.0, None, None) == binding.KVD_ERR_INVALID_ARG
    assert lib.kvd_decode_attention_recompute(None, 0, 0, None, None, None, None, None, 0, None, None, 0, None, 0, 0.0,
                                              None, None) == binding.KVD_ERR_INVALID_ARG
    assert lib.kvd_decode_attention_recompute_fp8(None, 0, 0, None, None, None, None, 0, 0, None, 0, 0.0, None,
                                                  None) == binding.KVD_ERR_INVALID_ARG
    # the allocation-free entry point validates shapes and limits on the host before it looks for a device
    qp = (ctypes.c_int32 * 1)(0)
    assert lib.kvd_decode_attention_static(8, 4, 96, 0, 1, None, qp, None, 0, 0.0, None, None) == binding.KVD_ERR_SHAPE
    assert lib.kvd_decode_attention_static(7, 4, 128, 0, 1, None, qp, None, 0, 0.0, None, None) == binding.KVD_ERR_SHAPE
    assert lib.kvd_decode_attention_static(8, 4, 128, -1, 1, None, qp, None, 0, 0.0, None, None) == binding.KVD_ERR_INVALID_ARG
    assert lib.kvd_decode_attention_static(8, 4, 128, 0, 0, None, None, None, 0, 0.0, None, None) == binding.KVD_OK  # empty batch
    assert lib.kvd_decode_attention_static(8, 4, 128, 0, 1, None, qp, None, 0, 0.0, None, None) == binding.KVD_ERR_INVALID_ARG


def test_fused_predicate_is_host_only_and_shape_aware():
    gemma = kvd.make_desc(34, 2560, 8, 4, 256, 1e-6, True, 1e-6)
    smol = kvd.make_desc(1, 576, 9, 3, 64, 1e-5, False, 1e-5)
    assert not kvd.kvd_fused_recompute_pays(gemma, 4096) and kvd.kvd_fused_recompute_pays(gemma, 32768)
    assert kvd.kvd_fused_recompute_pays(gemma, 4096, fp8=True) and not kvd.kvd_fused_recompute_pays(gemma, 1024, fp8=True)
    assert not kvd.kvd_fused_recompute_pays(smol, 1 << 20)  # no fused kernel for this shape
    assert not kvd.kvd_fused_recompute_pays(gemma, 0)
