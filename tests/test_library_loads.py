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
    header = open(os.path.join(ROOT, "include", "kvd.h")).read()
    declared = set(re.findall(r"\b(kvd_[a-z_0-9]+)\s*\(", header))
    declared -= {"kvd_ctx"}
    assert declared == set(binding.EXPORTED_SYMBOLS)
    for name in sorted(declared):
        assert hasattr(lib, name), name


def test_version_and_status_strings():
    assert kvd.kvd_version() == "0.1"
    assert kvd.status_string(0) == "ok"
    for s in range(1, 10):
        assert kvd.status_string(s) not in ("ok", "unknown status")


def test_size_queries_validate_shapes_without_a_device():
    good = kvd.make_desc(34, 2560, 8, 4, 256, 1e-6, True, 1e-6, max_seqs=2, max_tokens_per_seq=4096, max_batch=2)
    # rows + positions for 1 layer: 2 seqs * 4096 tokens * (2560 * 2 + 4) bytes
    assert kvd.kvd_store_bytes(good, 1) == 2 * 4096 * (2560 * 2 + 4)
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
