"""The multi-GPU mode of bench.py is N independent replicas (the hot path has no exchange step).
What N > 1 adds is the aggregation: the job's time is the slowest rank's, the value is the sum of
the units.  Checked here with two gloo ranks on CPU; the reference arm runs on rank 0 only."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
# rank 0 took 10 ms for 5 steps, rank 1 took 30 ms: the job is as slow as rank 1
ms_per_step, value = bench.aggregate_replicas(10.0 if rank == 0 else 30.0, 4096, 5, dist, "cpu")
with open(os.path.join({out!r}, "rank%d.json" % rank), "w") as f:
    json.dump({{"rank": rank, "ms_per_step": ms_per_step, "value": value}}, f)
dist.barrier()
dist.destroy_process_group()
"""


def test_two_gloo_ranks_aggregate_as_max_time_and_summed_units(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, out=str(tmp_path)))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29577", str(script)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    rows = [json.load(open(tmp_path / f"rank{r}.json")) for r in (0, 1)]
    assert sorted(r["rank"] for r in rows) == [0, 1]
    for r in rows:
        assert r["ms_per_step"] == pytest.approx(6.0)
        assert r["value"] == pytest.approx(2 * 4096 / 6.0e-3)


def test_single_process_aggregation():
    sys.path.insert(0, ROOT)
    import bench
    ms, v = bench.aggregate_replicas(8.0, 100, 4)
    assert ms == 2.0 and v == pytest.approx(100 / 2e-3)


def test_reference_arm_prints_the_contract_line_and_only_rank0_works():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=240, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""  # other ranks exit 0 without work
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    out = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    assert line["metric"] == "recomputed_kv_tokens_per_s" and line["unit"] == "tokens/s"
