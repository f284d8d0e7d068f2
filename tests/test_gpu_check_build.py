"""The checking build (libkvd_check.so, -DKVD_CHECK): the same kernels with device-side index tests.

A memory checker cannot be run on the machines this library is developed on, so the library carries its own
stand-in: a second build whose kernels test the indices they derive on the device (tile -> job and row block,
store-range rows, residual-row slots, attention-partial slots) and, instead of accessing out of range, set a
bit of the status word that kvd_poll_status reports as KVD_ERR_BOUNDS.

This test (1) shows the mechanism reporting, through the self-test entry point whose index is out of range by
construction and whose guarded access is skipped, and the context staying usable afterwards; (2) runs the
oracle-parity suites of the recompute, attention, fused and FP8 paths against the checking build in a child
process -- every one of those tests ends by polling the status word, so a failed index test anywhere fails it.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu

SELFTEST = r'''
import sys
sys.path.insert(0, "tests")
import numpy as np, torch
import paper_2603_19664_b200 as kvd
from paper_2603_19664_b200 import binding
from kvd_synth import TINY_GQA, make_residuals
from gpu_util import dev, host_f64, kv_errors, open_layer, oracle_kv
assert binding.LIB_PATH.endswith("libkvd_check.so") and binding.kvd_build_has_checks()
shape = TINY_GQA
ctx, w = open_layer(shape, max_tokens=512, with_store=True)
assert ctx.kvd_poll_status() == kvd.KVD_OK
assert ctx.kvd_selftest_bounds_check() == kvd.KVD_OK      # enqueued
assert ctx.kvd_poll_status() == binding.KVD_ERR_BOUNDS    # the failed index test is reported ...
assert ctx.kvd_poll_status() == kvd.KVD_OK                # ... once, and the word is clear again
# the context still works: a recompute through the checking build, against the oracle
T, kdim = 300, shape.n_kv_heads * shape.d_head
X = make_residuals(shape, T, seed=5)
pos = np.arange(T)
x, p = dev(X), torch.from_numpy(pos.astype(np.int32)).cuda()
ctx.kvd_checkpoint_residual(0, 0, x, p, T)
k = torch.empty((T, kdim), dtype=torch.bfloat16, device="cuda"); v = torch.empty_like(k)
ctx.kvd_recompute_kv(0, None, None, T, k, v, kdim, seq=0, first_row=0)
assert ctx.kvd_poll_status() == kvd.KVD_OK
Kr, Vr = oracle_kv(shape, w, X, pos)
for g, r in ((host_f64(k), Kr.reshape(T, kdim)), (host_f64(v), Vr.reshape(T, kdim))):
    mx, rel = kv_errors(g, r)
    assert mx <= 2e-2 and rel <= 1e-2
print("checking build ok")
'''


def test_checking_build_reports_and_passes_the_parity_suites():
    from paper_2603_19664_b200.build import build
    import paper_2603_19664_b200 as kvd
    build(check=True)
    assert not kvd.binding.kvd_build_has_checks() or os.environ.get("KVD_LIBRARY")  # this process runs the release build
    env = dict(os.environ, KVD_LIBRARY="check")
    r = subprocess.run([sys.executable, "-c", SELFTEST], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "checking build ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
    files = ["tests/test_gpu_recompute.py", "tests/test_gpu_attention.py", "tests/test_gpu_fused.py", "tests/test_gpu_fp8.py",
             "tests/test_gpu_scaffold.py"]
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider", *files], cwd=ROOT,
                       env=env, capture_output=True, text=True, timeout=1800)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout
