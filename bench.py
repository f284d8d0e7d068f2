#!/usr/bin/env python
"""Benchmark of the KV-Direct hot path on one B200 (or N independent replicas).

One *step* is one pass of the whole per-layer hot path over one batch of synthetic input, on a
single decoder layer shaped like Gemma-3-4B (hidden 2560, 8 query / 4 KV heads, head_dim 256,
key norm, RoPE base 1e6) with T = 4096 checkpointed tokens:

    kvd_checkpoint_residual (T rows)           STORE_RESIDUAL of Algorithm 1
    kvd_recompute_kv_step   (T rows from store  Eq. 13-14: RMSNorm -> [W_K|W_V] GEMM -> key norm -> RoPE,
                             + 1 new row)       and K_t, V_t of the current token, in one launch
    kvd_decode_attention    (T + 1 keys)        Eq. 6-7, query at position T

The JSON line printed by rank 0 follows the repository's bench contract; `value` is recomputed-KV
tokens per second over whole steps with inputs resident in HBM, `e2e` the same with host buffers and
the copies timed, `roofline` describes the recompute GEMM against the measured dense-bf16 peak,
`roofline_attention` the decode attention against the measured HBM copy bandwidth, `cached_read`
the thing KV-Direct replaces (attention over a stored cache, and a plain device copy of it), and
`cpu_baseline` the fp64 oracle timed on the host cores on a bounded sample.

`--impl reference` times the CPU oracle alone (there is no other reference implementation of the
paper's method to run).  `--sweep` adds the recompute-vs-read table over T = 256 .. 32768.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "recomputed_kv_tokens_per_s"
UNIT = "tokens/s"
T_TOKENS = 4096
DATASHEET_BF16_TFLOPS = 2250.0  # dense, NVIDIA's figure without sparsity
DATASHEET_HBM_GBS = 8000.0
N_SETS = 16  # rotating buffer sets: 16 x (21 MB residual rows + 21 MB store + 16.8 MB K/V) >> 126 MB of L2


def profile_traffic(filename, kernel_substring):
    """DRAM bytes (read + write) of one launch of a kernel, read from the ncu summary committed under
    profiles/ (the first launch whose header line contains `kernel_substring`).  Returns a dict with the
    bytes and the file they came from, or None entries if the file or the counters are not there."""
    path = os.path.join(ROOT, "profiles", filename)
    unit = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    got, inside = {}, False
    try:
        with open(path) as f:
            for line in f:
                if line.startswith("--- launch"):
                    if inside and len(got) == 2:
                        break
                    inside = kernel_substring in line
                    got = {}
                elif inside:
                    parts = line.split()
                    if len(parts) >= 4 and parts[0] in ("dram__bytes_read.sum", "dram__bytes_write.sum") and parts[3] in unit:
                        got[parts[0]] = float(parts[2]) * unit[parts[3]]
    except OSError:
        return {"bytes": None, "source": None}
    if len(got) != 2:
        return {"bytes": None, "source": None}
    return {"bytes": got["dram__bytes_read.sum"] + got["dram__bytes_write.sum"], "source": "profiles/" + filename}


def workload_config(n_sets, world):
    """The `config` object of the JSON line: the same keys and workload in both arms."""
    return {"workload": "gemma3-4b layer (d=2560, 8q/4kv heads, d_head=256, key norm, theta=1e6), "
                        "T=4096 checkpointed tokens, batch 1 (config 2)",
            "step": "checkpoint T rows -> recompute K/V of T rows from the store + K_t,V_t of the current "
                    "token (one launch) -> decode attention over T+1 keys",
            "l2": f"inputs rotate over {n_sets} buffer sets (~{n_sets * 59} MB), larger than L2",
            "launch": "steps replayed from CUDA graphs of the captured launch sequence",
            "replicas": "independent replicas per GPU, no collective" if world > 1 else "single GPU"}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.005)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------- CPU oracle timing
class OracleTimer:
    """Times the fp64 oracle (as it stands) on a bounded sample of one step's work."""

    def __init__(self, shape, T):
        import oracle
        from kvd_synth import bf16_to_f64, make_kv, make_layer_weights, make_query, make_residuals
        self.oracle, self.shape, self.T = oracle, shape, T
        w = make_layer_weights(shape)
        self.args = (bf16_to_f64(w.gamma_in), bf16_to_f64(w.w_kv), shape.n_kv_heads, shape.d_head, shape.rms_eps,
                     shape.rope_theta, bf16_to_f64(w.gamma_k) if w.gamma_k is not None else None, shape.rms_eps)
        self.cores = oracle.max_threads()
        self.X = bf16_to_f64(make_residuals(shape, T, seed=99, outliers=True))
        K, V = make_kv(shape, T + 1, seed=99)
        self.Kf, self.Vf = bf16_to_f64(K), bf16_to_f64(V)
        self.q = bf16_to_f64(make_query(shape, 1, seed=99))[0]
        t0 = time.perf_counter()
        self._recompute(16)
        self.s_per_row = (time.perf_counter() - t0) / 16  # calibration only

    def _recompute(self, rows):
        self.oracle.recompute_kv(self.X[:rows], np.arange(rows, dtype=np.int32), *self.args)

    def step(self, budget_s):
        """One bounded sample: recompute_kv on as many rows as fit the budget (16..T), then the
        attention over all T + 1 keys; the row part is scaled linearly to T rows (rows are independent)."""
        T = self.T
        rows = int(min(self.X.shape[0], max(16, budget_s * 0.8 / max(self.s_per_row, 1e-6)))) // 16 * 16
        t0 = time.perf_counter()
        self._recompute(rows)
        t_rec = time.perf_counter() - t0
        t0 = time.perf_counter()
        self.oracle.decode_attention(self.q, T, [(self.Kf, self.Vf, 0)], 1.0 / math.sqrt(self.shape.d_head), 0)
        t_att = time.perf_counter() - t0
        step_s = t_rec * T / rows + t_att
        return {"value": T / step_s, "unit": UNIT, "cores": self.cores, "kind": "oracle",
                "sample": f"recompute_kv on {rows} of {T} rows ({t_rec:.2f} s, scaled linearly to {T} rows) + "
                          f"decode_attention over all {T + 1} keys ({t_att * 1e3:.1f} ms)"}


def run_reference(args):
    from kvd_synth import GEMMA3_4B_GLOBAL
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    timer = OracleTimer(GEMMA3_4B_GLOBAL, T_TOKENS)
    budget = min(4.0, max(0.05, 150.0 / max(args.steps + args.warmup, 1)))
    for _ in range(args.warmup):
        timer.step(budget)
    vals, base = [], None
    t0 = time.perf_counter()
    for _ in range(args.steps):
        base = timer.step(budget)
        vals.append(base["value"])
    wall = time.perf_counter() - t0
    v = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * wall / max(args.steps, 1), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(args.sets, 1),
            "note": "each step times the fp64 CPU oracle on a bounded sample of the same workload and scales linearly "
                    "to T rows; the launch and L2 entries of config describe the GPU arm's run of it",
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": base["cores"], "kind": "oracle", "sample": base["sample"]},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- replicas
def aggregate_replicas(local_ms: float, units_per_rank: int, steps: int, dist=None, device="cpu"):
    """Whole-job throughput of independent replicas: every rank processed `units_per_rank` units per
    step; the job's time is the slowest rank's.  Returns (ms_per_step, units_per_second).  With
    `dist` = None this is the single-process case."""
    import torch
    world = 1
    if dist is not None:
        t = torch.tensor([local_ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        local_ms = float(t.item())
        world = dist.get_world_size()
    ms_per_step = local_ms / steps
    return ms_per_step, world * units_per_rank / (ms_per_step * 1e-3)


# ----------------------------------------------------------------------------- GPU arm
class GraphEvent:
    """A CUDA event that can be recorded inside a captured graph (an event-record node) and timed
    afterwards; torch's own events cannot be timed when recorded during capture."""

    def __init__(self):
        try:
            from cuda.bindings import runtime as rt
        except ImportError:  # older cuda-python layout
            from cuda import cudart as rt
        self.rt = rt
        err, self.e = rt.cudaEventCreate()
        assert int(err) == 0, err

    def record(self):
        import torch
        (err,) = self.rt.cudaEventRecordWithFlags(self.e, torch.cuda.current_stream().cuda_stream, 1)  # external
        assert int(err) == 0, err

    def elapsed_ms(self, other):
        err, ms = self.rt.cudaEventElapsedTime(self.e, other.e)
        assert int(err) == 0, err
        return ms


class Workload:
    """Device buffers and the step function for the Gemma-3-4B-shaped layer."""

    def __init__(self, shape, T, n_sets):
        import torch
        import paper_2603_19664_b200 as kvd
        from kvd_synth import make_layer_weights, make_query, make_residuals
        self.torch, self.kvd, self.shape, self.T, self.n_sets = torch, kvd, shape, T, n_sets
        self.kdim = shape.n_kv_heads * shape.d_head

        def dev(bits):
            return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

        w = make_layer_weights(shape)
        self.desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                                  shape.qk_norm, shape.rms_eps, shape.rope_style, n_sets, T + 8, 1)
        self.ctx = kvd.Kvd(self.desc)
        self.w_kv, self.g_in = dev(w.w_kv), dev(w.gamma_in)
        self.g_k = dev(w.gamma_k) if w.gamma_k is not None else None
        self.ctx.kvd_set_layer(0, self.w_kv, self.g_in, self.g_k, shape.rope_theta, shape.sliding_window)
        self.ws = torch.empty(kvd.kvd_workspace_bytes(self.desc), dtype=torch.uint8, device="cuda")
        self.ctx.kvd_attach_workspace(self.ws)
        self.arena = torch.empty(kvd.kvd_store_bytes(self.desc, 1), dtype=torch.uint8, device="cuda")
        self.ctx.kvd_attach_store(self.arena, 1)
        # the FP8 checkpoint variant's store (a second arena), filled once per set below
        self.arena8 = torch.empty(kvd.kvd_store_bytes_fp8(self.desc, 1), dtype=torch.uint8, device="cuda")
        self.ctx.kvd_attach_store_fp8(self.arena8, 1)
        # the FP4 checkpoint variant's store (a third arena) and the scratch its recompute expands rows into
        self.arena4 = torch.empty(kvd.kvd_store_bytes_fp4(self.desc, 1), dtype=torch.uint8, device="cuda")
        self.ctx.kvd_attach_store_fp4(self.arena4, 1)
        self.scratch4 = torch.empty(kvd.kvd_fp4_scratch_bytes(self.desc, T), dtype=torch.uint8, device="cuda")
        x_bits = make_residuals(shape, T + 1, seed=2, outliers=True)
        self.x_host_bits = x_bits
        x0 = dev(x_bits)
        # distinct memory per set, same distribution: rows rotated by a set-dependent offset
        self.X = [x0 if i == 0 else torch.roll(x0, shifts=97 * i, dims=0).contiguous() for i in range(n_sets)]
        self.pos = torch.arange(T + 1, dtype=torch.int32, device="cuda")
        self.K = [torch.empty((T + 1, self.kdim), dtype=torch.bfloat16, device="cuda") for _ in range(n_sets)]
        self.V = [torch.empty((T + 1, self.kdim), dtype=torch.bfloat16, device="cuda") for _ in range(n_sets)]
        self.q = dev(make_query(shape, n_sets, seed=2))  # one query per set
        self.out = torch.empty((n_sets, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16, device="cuda")
        self.ev = None

    def step(self, i, events=None):
        """One pass of the hot path on buffer set i % n_sets.  `events` (optional): 4 CUDA events
        recorded around checkpoint / recompute (stored rows + current token) / attention."""
        s, T, c = i % self.n_sets, self.T, self.ctx
        X, K, V = self.X[s], self.K[s], self.V[s]
        c.kvd_reset_sequence(s)
        if events:
            events[0].record()
        c.kvd_checkpoint_residual(s, 0, X, self.pos, T)
        if events:
            events[1].record()
        # one launch: K/V of the T stored rows and (K_t, V_t) of the current token
        c.kvd_recompute_kv_step(0, [(s, 0, T, K, V)], X[T:], self.pos[T:], 1, K[T:], V[T:], self.kdim)
        if events:
            events[2].record()
        c.kvd_decode_attention(0, 1, self.q[s:s + 1], [T],
                               [[(K, V, self.kdim, 0, T), (K[T:], V[T:], self.kdim, T, 1)]], 0.0, self.out[s:s + 1])
        if events:
            events[3].record()

    # the launches of a step, individually (for per-kernel timing)
    def k_checkpoint(self, i):
        s = i % self.n_sets
        self.ctx.kvd_reset_sequence(s)
        self.ctx.kvd_checkpoint_residual(s, 0, self.X[s], self.pos, self.T)

    def k_recompute(self, i):
        # RECOMPUTE_KV of Algorithm 1: T checkpointed rows of set s (filled by the last step on it)
        s = i % self.n_sets
        self.ctx.kvd_recompute_kv(0, None, None, self.T, self.K[s], self.V[s], self.kdim, seq=s, first_row=0)

    def k_recompute_rows(self, i):
        # the same rows handed over by the caller instead (a prefill-shaped call: their statistics are
        # taken by a small kernel of their own first, two launches)
        s = i % self.n_sets
        self.ctx.kvd_recompute_kv(0, self.X[s], self.pos, self.T, self.K[s], self.V[s], self.kdim)

    def k_recompute_step(self, i):
        # the step's launch: T rows from the store of set s (filled by the last step on it) + 1 new row
        s, T = i % self.n_sets, self.T
        self.ctx.kvd_recompute_kv_step(0, [(s, 0, T, self.K[s], self.V[s])], self.X[s][T:], self.pos[T:], 1,
                                       self.K[s][T:], self.V[s][T:], self.kdim)

    def k_current(self, i):
        s, T = i % self.n_sets, self.T
        self.ctx.kvd_recompute_kv(0, self.X[s][T:], self.pos[T:], 1, self.K[s][T:], self.V[s][T:], self.kdim)

    def k_attention(self, i):
        s, T = i % self.n_sets, self.T
        K, V = self.K[s], self.V[s]
        self.ctx.kvd_decode_attention(0, 1, self.q[s:s + 1], [T],
                                      [[(K, V, self.kdim, 0, T), (K[T:], V[T:], self.kdim, T, 1)]], 0.0,
                                      self.out[s:s + 1])

    def k_checkpoint_fp8(self, i):
        s = i % self.n_sets
        self.ctx.kvd_reset_sequence_fp8(s)
        self.ctx.kvd_checkpoint_residual_fp8(s, 0, self.X[s], self.pos, self.T)

    def k_recompute_fp8(self, i):
        # RECOMPUTE_KV from E4M3 checkpoints (rows and weights as FP8 codes, tensor-core kind f8f6f4)
        s = i % self.n_sets
        self.ctx.kvd_recompute_kv_fp8(0, [(s, 0, self.T, self.K[s], self.V[s])], self.kdim)

    def k_checkpoint_fp4(self, i):
        s = i % self.n_sets
        self.ctx.kvd_reset_sequence_fp4(s)
        self.ctx.kvd_checkpoint_residual_fp4(s, 0, self.X[s], self.pos, self.T)

    def k_recompute_fp4(self, i):
        # RECOMPUTE_KV from FP4 checkpoints: rows expanded to bf16 (exactly) into a scratch, then the bf16 projection
        s = i % self.n_sets
        self.ctx.kvd_recompute_kv_fp4(0, [(s, 0, self.T, self.K[s], self.V[s])], self.kdim, self.scratch4)

    def k_two_call(self, i):
        # recompute (T stored rows + the current token) followed by attention: the step's two K/V launches
        self.k_recompute_step(i)
        self.k_attention(i)

    def k_fused(self, i):
        # the same work with the recomputed K/V consumed inside the recompute kernel (never written):
        # kvd_decode_attention_recompute; only the current token's K_t, V_t are stored and read back
        s, T = i % self.n_sets, self.T
        K, V = self.K[s], self.V[s]
        self.ctx.kvd_decode_attention_recompute(0, 1, self.q[s:s + 1], [T], [(s, 0, T)], self.X[s][T:], self.pos[T:], 1,
                                                K[T:], V[T:], self.kdim, [[(K[T:], V[T:], self.kdim, T, 1)]], 0.0,
                                                self.out[s:s + 1])

    def append_current(self):
        # the current token's row joins the bf16 store of every set (row T), once, outside any timed region
        for s in range(self.n_sets):
            if self.ctx.kvd_rows_stored(0, s) == self.T:
                self.ctx.kvd_checkpoint_residual(s, 0, self.X[s][self.T:], self.pos[self.T:], 1)

    def k_fused_folded(self, i):
        # the fused call with the current token inside the attended range (its row is checkpointed like every
        # token's): no live segment is left, so the streaming launch disappears -- recompute+attend, merge.
        # K_t, V_t are still written (the caller's row rides in the same launch) for a window that keeps them.
        s, T = i % self.n_sets, self.T
        K, V = self.K[s], self.V[s]
        self.ctx.kvd_decode_attention_recompute(0, 1, self.q[s:s + 1], [T], [(s, 0, T + 1)], self.X[s][T:], self.pos[T:], 1,
                                                K[T:], V[T:], self.kdim, [[]], 0.0, self.out[s:s + 1])

    def append_current_fp8(self):
        # the current token joins the FP8 store of every set (row T), once, outside any timed region
        for s in range(self.n_sets):
            if self.ctx.kvd_rows_stored_fp8(0, s) == self.T:
                self.ctx.kvd_checkpoint_residual_fp8(s, 0, self.X[s][self.T:], self.pos[self.T:], 1)

    def k_two_call_fp8(self, i):
        # nothing kept: K/V of all T + 1 tokens rebuilt from their FP8 checkpoints, then attention over them
        s, T = i % self.n_sets, self.T
        K, V = self.K[s], self.V[s]
        self.ctx.kvd_recompute_kv_fp8(0, [(s, 0, T + 1, K, V)], self.kdim)
        self.ctx.kvd_decode_attention(0, 1, self.q[s:s + 1], [T], [[(K, V, self.kdim, 0, T + 1)]], 0.0,
                                      self.out[s:s + 1])

    def k_fused_fp8(self, i):
        # the same with the rebuilt K/V consumed inside the recompute kernel: kvd_decode_attention_recompute_fp8
        s, T = i % self.n_sets, self.T
        self.ctx.kvd_decode_attention_recompute_fp8(0, 1, self.q[s:s + 1], [T], [(s, 0, T + 1)], [], self.kdim, [[]],
                                                    0.0, self.out[s:s + 1])

    def cached_read_step(self, i):
        """What KV-Direct replaces: attention over the stored cache of T + 1 keys in one segment."""
        s, T = i % self.n_sets, self.T
        self.ctx.kvd_decode_attention(0, 1, self.q[s:s + 1], [T], [[(self.K[s], self.V[s], self.kdim, 0, T + 1)]],
                                      0.0, self.out[s:s + 1])


def run_gpu(args):
    import torch
    from kvd_synth import GEMMA3_4B_GLOBAL
    import paper_2603_19664_b200 as kvd
    from paper_2603_19664_b200.build import build
    build()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_mod

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    shape, T = GEMMA3_4B_GLOBAL, T_TOKENS
    peaks = load_peaks()
    n_sets = args.sets
    wl = Workload(shape, T, n_sets)
    steps, warmup = args.steps, max(args.warmup, 3)

    # ---- warm-up (eager launches)
    for i in range(warmup):
        wl.step(i)
    barrier()
    assert wl.ctx.kvd_poll_status() == kvd.KVD_OK

    if args.profile:
        # plain eager launches for a profiler: no graphs, no auxiliary measurements
        for i in range(steps):
            wl.step(warmup + i)
        # the FP8 checkpoint variant of the same layer: quantising checkpoint + recompute, two sets
        for i in range(2):
            wl.k_checkpoint_fp8(i)
            wl.k_recompute_fp8(i)
        # and the FP8 checkpoints rebuilt and attended in one kernel (T + 1 rows, nothing kept)
        wl.append_current_fp8()
        for i in range(2):
            wl.k_fused_fp8(i)
        barrier()
        if args.profile_long_attn:
            # a few eager decode-attention calls over 32769 keys (134 MB each, larger than L2)
            def eager(fn, reps):
                for i in range(3):
                    fn(i)
                torch.cuda.synchronize()
                return 1.0  # not a measurement
            measure_long_attention(wl, peaks, eager)
        if args.profile_prefill_attn:
            # a few causal prefill-attention calls over 4096 tokens of the layer
            measure_prefill_attention(wl, peaks, lengths=(4096,))
        if rank == 0:
            print(json.dumps({"profile_run": True, "steps": steps, "launches": wl.ctx.kvd_launch_count()}))
        return

    # ---- the step is a fixed launch sequence: capture it once per buffer set into CUDA graphs
    side = torch.cuda.Stream()

    def capture(n, events=None):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for i in range(n):
                wl.step(i, events[i] if events else None)
        return g

    l0 = wl.ctx.kvd_launch_count()
    g_full = capture(n_sets)
    launches_per_step = (wl.ctx.kvd_launch_count() - l0) // n_sets
    g_rem = capture(steps % n_sets) if steps % n_sets else None
    kev = [[GraphEvent() for _ in range(4)] for _ in range(n_sets)]
    g_ev = capture(n_sets, kev)
    for _ in range(2):
        g_full.replay()
    barrier()

    # ---- timed region: exactly `steps` steps between two events, repeated until at least ~0.3 s of GPU time
    # has been timed (a single pass of a 50 us step is over before the clocks can be sampled twice); the
    # median repeat is reported
    def timed_pass():
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps // n_sets):
            g_full.replay()
        if g_rem is not None:
            g_rem.replay()
        b.record()
        return a, b
    barrier()
    a0, b0 = timed_pass()
    barrier()
    first_ms = a0.elapsed_time(b0)
    n_rep = int(min(2000, max(5, math.ceil(300.0 / max(first_ms, 1e-3)))))
    with ClockSampler(local) as clocks:
        barrier()
        passes = [timed_pass() for _ in range(n_rep)]
        barrier()
        rep_ms = np.array([a.elapsed_time(b) for a, b in passes])
        # per-kernel durations: the same steps with event-record nodes between the kernels
        t_k = [[], [], []]
        for _ in range(max(2, min(20, steps // n_sets))):
            g_ev.replay()
            torch.cuda.synchronize()
            for e in kev:
                for j in range(3):
                    t_k[j].append(e[j].elapsed_ms(e[j + 1]))
    launches = launches_per_step * steps  # of the timed region (every repeat launches as many)
    total_ms = float(np.median(rep_ms))
    status = wl.ctx.kvd_poll_status()
    if status != kvd.KVD_OK:
        raise RuntimeError(f"device status after the timed region: {kvd.status_string(status)}")
    t_ckpt, t_gemm, t_attn = (np.array(t) for t in t_k)
    ms_per_step, value = aggregate_replicas(total_ms, T, steps, dist, "cuda")

    # ---- the read that recomputation replaces (graphs of n_sets calls, same rotation)
    def timed_graph(fn, reps):
        for i in range(n_sets):
            fn(i)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for i in range(n_sets):
                fn(i)
        g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (reps * n_sets)

    def timed(fn, n):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(n):
            fn(3 + i)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    # each kernel of the step on its own: a graph of n_sets back-to-back launches on rotating buffer
    # sets between two CUDA events (launch gaps included), averaged per launch
    iso_ms = {"checkpoint": timed_graph(wl.k_checkpoint, 10), "recompute": timed_graph(wl.k_recompute, 10),
              "recompute_with_current_token": timed_graph(wl.k_recompute_step, 10),
              "recompute_from_caller_rows": timed_graph(wl.k_recompute_rows, 10),
              "current_token_kv_alone": timed_graph(wl.k_current, 10), "attention": timed_graph(wl.k_attention, 10),
              "checkpoint_fp8": timed_graph(wl.k_checkpoint_fp8, 10),
              "checkpoint_fp4": timed_graph(wl.k_checkpoint_fp4, 10),
              "recompute_from_fp4_checkpoints": timed_graph(wl.k_recompute_fp4, 10),
              "recompute_from_fp8_checkpoints": timed_graph(wl.k_recompute_fp8, 10),
              "recompute_then_attention_two_calls": timed_graph(wl.k_two_call, 10),
              "recompute_fused_into_attention": timed_graph(wl.k_fused, 10)}
    wl.append_current()
    iso_ms["recompute_fused_into_attention_current_token_in_range"] = timed_graph(wl.k_fused_folded, 10)
    wl.append_current_fp8()
    iso_ms["recompute_fp8_then_attention_two_calls"] = timed_graph(wl.k_two_call_fp8, 10)
    iso_ms["recompute_fp8_fused_into_attention"] = timed_graph(wl.k_fused_fp8, 10)
    read_attn_ms = timed_graph(wl.cached_read_step, 10)
    # SM clock inside the recompute kernel: one traced launch, cycles over nanoseconds of CTA 0
    sm_mhz_in_kernel = None
    try:
        tr_buf = torch.zeros((148, 8, 16), dtype=torch.int64, device="cuda")
        wl.ctx.kvd_set_trace(tr_buf)
        mhz = []
        for i in range(6):
            wl.k_recompute(i)
            torch.cuda.synchronize()
            t0 = tr_buf[0, 0].cpu().numpy()
            if t0[13] > t0[12]:
                mhz.append(float(t0[14] - t0[11]) / float(t0[13] - t0[12]) * 1e3)
        wl.ctx.kvd_set_trace(None)
        sm_mhz_in_kernel = float(np.median(mhz[1:])) if len(mhz) > 1 else None
    except Exception:  # the trace hook is a diagnostic; the bench line does not depend on it
        sm_mhz_in_kernel = None
    kv_copy_dst = torch.empty((2, T + 1, wl.kdim), dtype=torch.bfloat16, device="cuda")

    def copy_step(i):
        s = i % wl.n_sets
        kv_copy_dst[0].copy_(wl.K[s])
        kv_copy_dst[1].copy_(wl.V[s])

    read_copy_ms = timed_graph(copy_step, 10)

    # ---- end to end through the C ABI with host buffers
    x_pin = torch.from_numpy(wl.x_host_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    pos_pin = torch.arange(T + 1, dtype=torch.int32).pin_memory()
    q_pin = wl.q[:1].cpu().pin_memory()
    out_pin = torch.empty((1, shape.n_q_heads, shape.d_head), dtype=torch.bfloat16).pin_memory()
    x_dev = [torch.empty_like(wl.X[0]) for _ in range(2)]
    pos_dev = [torch.empty_like(wl.pos) for _ in range(2)]
    q_dev = [torch.empty_like(wl.q[:1]) for _ in range(2)]
    out_dev = torch.empty_like(wl.out[:1])
    # Every step copies its own inputs from pinned host memory and its result back.  The copies of
    # step i + 1 are issued on a second stream while step i computes (two device buffers), as a serving
    # loop would do; the result of every step is still read by the host before the next step is launched.
    copy_stream = torch.cuda.Stream()
    ready = [torch.cuda.Event() for _ in range(2)]   # inputs of the step using buffer b have arrived
    freed = [torch.cuda.Event() for _ in range(2)]   # the step that used buffer b has consumed it
    issued = {}

    def issue_inputs(i):
        b = i % 2
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(freed[b])
            x_dev[b].copy_(x_pin, non_blocking=True)
            pos_dev[b].copy_(pos_pin, non_blocking=True)
            q_dev[b].copy_(q_pin, non_blocking=True)
            ready[b].record(copy_stream)
        issued[i] = True

    def e2e_step(i):
        s, b = i % wl.n_sets, i % 2
        cur = torch.cuda.current_stream()
        if i not in issued:
            issue_inputs(i)
        issue_inputs(i + 1)  # the next step's inputs travel while this step computes
        cur.wait_event(ready[b])
        xd, pd = x_dev[b], pos_dev[b]
        c = wl.ctx
        c.kvd_reset_sequence(s)
        c.kvd_checkpoint_residual(s, 0, xd, pd, T)
        c.kvd_recompute_kv_step(0, [(s, 0, T, wl.K[s], wl.V[s])], xd[T:], pd[T:], 1, wl.K[s][T:], wl.V[s][T:], wl.kdim)
        c.kvd_decode_attention(0, 1, q_dev[b], [T], [[(wl.K[s], wl.V[s], wl.kdim, 0, T), (wl.K[s][T:], wl.V[s][T:], wl.kdim, T, 1)]],
                               0.0, out_dev)
        freed[b].record(cur)
        out_pin.copy_(out_dev, non_blocking=True)
        cur.synchronize()  # the caller reads the result of every step
        issued.pop(i, None)

    def e2e_step_serial(i):
        # the same step with its copies on the computing stream (no overlap), for comparison
        s, b = i % wl.n_sets, i % 2
        x_dev[b].copy_(x_pin, non_blocking=True)
        pos_dev[b].copy_(pos_pin, non_blocking=True)
        q_dev[b].copy_(q_pin, non_blocking=True)
        xd, pd = x_dev[b], pos_dev[b]
        c = wl.ctx
        c.kvd_reset_sequence(s)
        c.kvd_checkpoint_residual(s, 0, xd, pd, T)
        c.kvd_recompute_kv_step(0, [(s, 0, T, wl.K[s], wl.V[s])], xd[T:], pd[T:], 1, wl.K[s][T:], wl.V[s][T:], wl.kdim)
        c.kvd_decode_attention(0, 1, q_dev[b], [T], [[(wl.K[s], wl.V[s], wl.kdim, 0, T), (wl.K[s][T:], wl.V[s][T:], wl.kdim, T, 1)]],
                               0.0, out_dev)
        out_pin.copy_(out_dev, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    n_e2e = min(max(steps, 10), 50)
    e2e_serial_ms = timed(e2e_step_serial, n_e2e)
    torch.cuda.synchronize()
    e2e_ms = timed(e2e_step, n_e2e)
    torch.cuda.synchronize()
    e2e_ms, _ = aggregate_replicas(e2e_ms, T, 1, dist, "cuda")
    h2d = x_pin.numel() * 2 + pos_pin.numel() * 4 + q_pin.numel() * 2
    d2h = out_pin.numel() * 2

    long_attn = measure_long_attention(wl, peaks, timed_graph) if rank == 0 else None
    prefill_attn = measure_prefill_attention(wl, peaks) if rank == 0 else None
    stack_decode = None
    if rank == 0 and world == 1 and not args.no_stack:
        stack_decode = measure_stack_decode((1, 4, 16, 64) if args.stack_all else (1, 4),
                                            **({"session_turns": 3, "session_gen": 16, "seg": (256, 512)} if args.short_session else {}))
    sweep = run_sweep(wl, peaks) if args.sweep and rank == 0 else None

    if rank == 0:
        flops = 4.0 * T * shape.n_kv_heads * shape.d_hidden * shape.d_head  # Eq. 26
        gemm_ms = iso_ms["recompute"]
        attn_ms = iso_ms["attention"]
        attn_bytes = (T + 1) * 4 * shape.n_kv_heads * shape.d_head  # Eq. 27 for T + 1 keys
        cpu = OracleTimer(shape, T).step(12.0)
        clk = clocks.summary()
        traffic_gemm = profile_traffic("recompute_kernel_gemma3_4b_t4096.txt", "kvd_recompute_kernel")
        traffic_attn = profile_traffic("attention_kernels_gemma3_4b_t4096.txt", "kvd_attn_split_kernel")
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": workload_config(n_sets, world),
            "clocks": clk,
            "repeats": {"n": len(rep_ms), "ms_per_step_median": float(np.median(rep_ms)) / steps,
                        "ms_per_step_min": float(np.min(rep_ms)) / steps, "ms_per_step_max": float(np.max(rep_ms)) / steps,
                        "timed_gpu_seconds": float(np.sum(rep_ms)) * 1e-3,
                        "note": "the region of exactly `steps` steps is timed `n` times back to back; value and "
                                "ms_per_step are the median repeat (max over ranks)",
                        "ms_per_step_x_sm_mhz": (float(np.median(rep_ms)) / steps * clk["sm_mhz"]) if clk.get("sm_mhz") else None},
            "e2e": {"value": world * T / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "ms_per_step_copies_not_overlapped": e2e_serial_ms,
                    "note": "every step copies its inputs from pinned host memory and its result back; the copies of "
                            "step i+1 run on a second stream under step i's kernels; PCIe-bound (21 MB per step)"},
            "gpu_launches": int(launches),
            "roofline": {"kernel": "kvd_recompute_kernel<256,256>", "bound": "tensor",
                         "achieved": flops / (gemm_ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": flops / (gemm_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                         # dram__bytes_read.sum + dram__bytes_write.sum of one launch, read from the ncu summary
                         "traffic": traffic_gemm["bytes"], "traffic_source": traffic_gemm["source"],
                         "algorithmic_bytes": 2 * (T * shape.d_hidden +
                         shape.d_hidden * shape.n_kv_cols + T * shape.n_kv_cols),
                         "peak_source": peaks["source"] + " burst", "avg_launch_us": gemm_ms * 1e3,
                         "in_step_us": float(np.mean(t_gemm)) * 1e3,
                         "timing": "graph of back-to-back launches on rotating inputs, CUDA events, per launch",
                         "frac_of_sustained": flops / (gemm_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                         "frac_of_datasheet": flops / (gemm_ms * 1e-3) / 1e12 / DATASHEET_BF16_TFLOPS,
                         "frac_in_step": flops / (float(np.mean(t_gemm)) * 1e-3) / 1e12 / peaks["bf16_tflops"],
                         "sm_mhz_in_kernel": sm_mhz_in_kernel,
                         "sm_mhz_note": "SM clock inside the kernel (clock64 against globaltimer over one traced launch); "
                                        "NVML samples taken between launches read higher"},
            # the FP8 checkpoint variant of the same launch: same flop count, E4M3 operands; its peak is the
            # measured bf16 peak times the nominal fp8 : bf16 ratio of 2 (no fp8 GEMM was measured on this machine)
            "roofline_fp8": {"kernel": "kvd_recompute_kernel<256,256,...,EB=1> (E4M3 rows and weights)", "bound": "tensor",
                             "achieved": flops / (iso_ms["recompute_from_fp8_checkpoints"] * 1e-3) / 1e12,
                             "peak": 2 * peaks["bf16_tflops"], "unit": "TFLOP/s",
                             "frac": flops / (iso_ms["recompute_from_fp8_checkpoints"] * 1e-3) / 1e12 / (2 * peaks["bf16_tflops"]),
                             "peak_source": peaks["source"] + " bf16 burst x 2 (nominal fp8 ratio)",
                             "avg_launch_us": iso_ms["recompute_from_fp8_checkpoints"] * 1e3,
                             "checkpoint_bytes_per_token": shape.d_hidden + 12, "traffic": None},
            "fp4_checkpoints": {"checkpoint_bytes_per_token": shape.d_hidden // 2 + shape.d_hidden // 16 + 12,
                                "bf16_checkpoint_bytes_per_token": 2 * shape.d_hidden + 8,
                                "kv_bytes_per_token_replaced": 4 * shape.n_kv_heads * shape.d_head,
                                "checkpoint_us": iso_ms["checkpoint_fp4"] * 1e3,
                                "recompute_us": iso_ms["recompute_from_fp4_checkpoints"] * 1e3,
                                "note": "E2M1 codes, E4M3 block scales per 16 channels, power-of-two row scale; rows are "
                                        "expanded to bf16 exactly and projected by the bf16 kernel (two launches)"},
            "roofline_attention": {"kernel": "kvd_attn_split_kernel<256,2> + merge", "bound": "hbm",
                                   "achieved": attn_bytes / (attn_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                                   "unit": "GB/s", "frac": attn_bytes / (attn_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                   "traffic": traffic_attn["bytes"], "traffic_source": traffic_attn["source"],
                                   "frac_of_datasheet": attn_bytes / (attn_ms * 1e-3) / 1e9 / DATASHEET_HBM_GBS,
                                   "avg_us": attn_ms * 1e3, "in_step_us": float(np.mean(t_attn)) * 1e3,
                                   "note": "16.8 MB per call: launch-latency bound; see attention_long"},
            "attention_long": long_attn,
            "prefill_attention": prefill_attn,
            "decode_step_us": {"total": ms_per_step * 1e3,
                               "isolated": {k: v * 1e3 for k, v in iso_ms.items()},
                               "in_step_with_event_nodes": {"checkpoint": float(np.mean(t_ckpt)) * 1e3,
                                                            "recompute_with_current_token": float(np.mean(t_gemm)) * 1e3,
                                                            "attention": float(np.mean(t_attn)) * 1e3}},
            "cached_read": {"attention_over_stored_cache_us": read_attn_ms * 1e3,
                            "attention_gbs": attn_bytes / (read_attn_ms * 1e-3) / 1e9,
                            "device_copy_us": read_copy_ms * 1e3,
                            "device_copy_gbs": 2 * attn_bytes / (read_copy_ms * 1e-3) / 1e9,
                            "recompute_over_read_ratio": gemm_ms / read_copy_ms,
                            "paper_ratio_context": "0.17-0.3x at N=500 on Apple M3 Max / MLX (paper Section 5.8)"},
            "cpu_baseline": {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")},
        }
        if stack_decode is not None:
            line["stack_decode_step"] = stack_decode
        if sweep is not None:
            line["sweep"] = sweep
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def measure_stack_decode(batches, n_check_steps=4, session_turns=20, session_gen=128, seg=(256, 1024)):
    """Configs 3 and 5 on the whole 34-layer Gemma-3-4B-shaped stack, nothing multiplied: a decode step of
    `batch` sequences with 2048 tokens of context behind them and a 256-token window, KV-Direct arm against
    full-cache arm from one shared state (tests/stack_harness.py: BatchStack).  Every kernel on the path is
    the library's (hot path through include/kvd.h, the rest of the block through include/kvd_scaffold.h).
    The step is captured into a CUDA graph and replayed; the hot path is also timed alone (same launches
    without the scaffold) so that the scaffold's share is visible.  Tokens of the two arms over
    `n_check_steps` greedy steps must be identical.  Then the config-5 session (full-size stack, `session_turns`
    turns of a user segment of seg[0]..seg[1] random tokens + `session_gen` greedy tokens, run once per cache
    policy) checks the token match through prefill and decode and reports the memory held."""
    import torch
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from kvd_synth import GEMMA3_4B_STACK
    from stack_harness import BatchStack, torch_stack_weights
    from session_config5 import run_session
    stack, ctx_len, window = GEMMA3_4B_STACK, 2048, 256
    w = torch_stack_weights(stack, seed=3)
    side = torch.cuda.Stream()
    rows = []
    for batch in batches:
        m = BatchStack(stack, w, batch, ctx_len, window, max_steps=n_check_steps)
        first = [(7919 * (b + 1)) % stack.vocab for b in range(batch)]
        tok_full = m.decode(first, n_check_steps, "full")
        tok_kvd = m.decode(first, n_check_steps, "kvdirect")
        tok = torch.tensor(first, dtype=torch.int32, device="cuda")
        rec = {"batch": batch, "tokens_match": tok_full == tok_kvd, "steps_compared": n_check_steps,
               "distinct_tokens": len({t for r in tok_full for t in r})}
        for policy in ("full", "kvdirect"):
            for scaffold in (True, False):
                l0 = m.ctx.kvd_launch_count()
                m.step(tok, ctx_len, policy, scaffold)
                launches = m.ctx.kvd_launch_count() - l0
                torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    m.step(tok, ctx_len, policy, scaffold)
                g.replay()
                torch.cuda.synchronize()
                time.sleep(0.2)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                reps = 10
                a.record()
                for _ in range(reps):
                    g.replay()
                b.record()
                torch.cuda.synchronize()
                key = ("kvdirect" if policy == "kvdirect" else "fullcache") + ("_step_us" if scaffold else "_hot_path_us")
                rec[key] = a.elapsed_time(b) / reps * 1e3
                if scaffold:
                    rec[key.replace("_step_us", "_kernel_launches")] = int(launches)
                del g
        rec["scaffold_us"] = rec["fullcache_step_us"] - rec["fullcache_hot_path_us"]
        rec["hot_path_ratio_kvdirect_over_fullcache"] = rec["kvdirect_hot_path_us"] / rec["fullcache_hot_path_us"]
        n_old = 5 * (ctx_len - window) + 29 * max(0, 1024 - 1 - window)
        rec["rows_recomputed_per_step"] = batch * n_old
        rec["recomputed_token_layers_per_s"] = batch * n_old / (rec["kvdirect_hot_path_us"] * 1e-6)
        assert m.ctx.kvd_poll_status() == 0
        m.ctx.close()
        del m
        torch.cuda.empty_cache()
        rows.append(rec)
    # ---- prefill of a whole segment through the stack: STORE_RESIDUAL and K/V of every layer, attention of all tokens
    # to themselves in one tcgen05 launch per layer (kvd_prefill_attention), the block's products at M = segment length
    from stack_harness import GpuStack
    from kvd_synth import make_token_ids
    prefill = []
    for U in (2048, 8192):
        g = GpuStack(stack, w, policy="full", max_tokens=U + 8, device_weights=True, tiled_attention=True)
        toks = make_token_ids(U, stack.vocab, seed=11).tolist()
        g.prefill(toks)  # warm-up at full size: first launches of every kernel, the allocator's blocks
        g.ctx.kvd_reset_sequence(0)
        g.t = 0
        torch.cuda.synchronize()
        l0, t0 = g.ctx.kvd_launch_count(), time.perf_counter()
        g.prefill(toks)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        assert g.ctx.kvd_poll_status() == 0
        prefill.append({"tokens": U, "ms": dt * 1e3, "tokens_per_s": U / dt, "kernel_launches": int(g.ctx.kvd_launch_count() - l0),
                        "timing": "host clock around the eager launches and a synchronize"})
        g.ctx.close()
        del g
        torch.cuda.empty_cache()
    t_session = time.perf_counter()
    recs, ok = run_session(stack, w, session_turns, session_gen, window, seg[0], seg[1],
                           session_turns * (seg[1] + session_gen) + 8)
    session = {"stack": stack.name, "turns": session_turns, "generated_per_turn": session_gen, "window": window,
               "user_segment_tokens": [r["user_tokens"] for r in recs], "tokens_total": recs[-1]["tokens_so_far"],
               "all_tokens_match": bool(ok), "peak_full_cache_kv_bytes": max(r["full_cache_kv_bytes"] for r in recs),
               "peak_kvdirect_live_kv_bytes": max(r["kvdirect_live_kv_bytes"] for r in recs),
               "rows_recomputed": recs[-1]["rows_recomputed_so_far"],
               "final_per_layer_checkpoint_bytes": recs[-1]["kvdirect_checkpoint_bytes_per_layer_rows"],
               "eq28_bytes_single_checkpoint_accounting": recs[-1]["kvdirect_eq28_bytes_single_checkpoint_accounting"],
               "last_turn_seconds_full_cache": recs[-1]["seconds_full_cache"],
               "last_turn_seconds_kvdirect": recs[-1]["seconds_kvdirect"],
               "wall_seconds_both_arms": time.perf_counter() - t_session,
               "note": "config 5 of BASELINE.json on the full-size stack; python tests/session_config5.py prints it per turn"}
    return {"config3_gemma3_4b_stack_ctx2048_window256": rows, "stack_prefill": prefill, "config5_session": session,
            "note": "34 layers, every launch measured (CUDA graph of one whole decode step, 10 replays); "
                    "scaffold = the block's other products and small steps on the library's own kernels"}


def run_profile_stack(args):
    """Eager launches of two whole-stack decode steps per cache policy (34 layers, batch 4, context 2048, window 256)
    for a run under a profiler: every kernel of the measured config-3 step, hot path and scaffold."""
    import torch
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from kvd_synth import GEMMA3_4B_STACK
    from stack_harness import BatchStack, torch_stack_weights
    from paper_2603_19664_b200.build import build
    build()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    w = torch_stack_weights(GEMMA3_4B_STACK, seed=3)
    m = BatchStack(GEMMA3_4B_STACK, w, 4, 2048, 256, max_steps=8)
    tok = torch.tensor([5, 6, 7, 8], dtype=torch.int32, device="cuda")
    for policy in ("full", "kvdirect"):
        for i in range(2):
            m.step(tok, 2048 + i, policy)
    torch.cuda.synchronize()
    assert m.ctx.kvd_poll_status() == 0
    print(json.dumps({"profile_run": "stack", "launches": m.ctx.kvd_launch_count()}))


def measure_long_attention(wl, peaks, timed_graph, T=32768):
    """Decode attention over T + 1 keys of the same layer shape (134 MB per call): the size at which
    the HBM roofline, not launch latency, is the bound."""
    import torch
    import paper_2603_19664_b200 as kvd
    shape, kdim = wl.shape, wl.kdim
    desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                         shape.qk_norm, shape.rms_eps, shape.rope_style, 1, T + 8, 1)
    ctx = kvd.Kvd(desc)
    ctx.kvd_set_layer(0, wl.w_kv, wl.g_in, wl.g_k, shape.rope_theta, 0)
    ws = torch.empty(kvd.kvd_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_workspace(ws)
    n = min(wl.n_sets, 5)
    K = [torch.randn((T + 1, kdim), device="cuda", dtype=torch.float32).to(torch.bfloat16) for _ in range(n)]
    V = [torch.randn((T + 1, kdim), device="cuda", dtype=torch.float32).to(torch.bfloat16) for _ in range(n)]

    def call(i):
        j = i % n
        ctx.kvd_decode_attention(0, 1, wl.q[:1], [T], [[(K[j], V[j], kdim, 0, T + 1)]], 0.0, wl.out[:1])

    ms = timed_graph(call, 5)
    byts = (T + 1) * 4 * shape.n_kv_heads * shape.d_head
    ctx.close()
    tr = profile_traffic("attention_kernel_gemma3_4b_t32768.txt", "kvd_attn_split_kernel")
    return {"keys": T + 1, "bytes": byts, "avg_us": ms * 1e3, "achieved": byts / (ms * 1e-3) / 1e9,
            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": byts / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "bound": "hbm", "kernel": "kvd_attn_split_kernel<256,2,4>",
            "frac_of_datasheet": byts / (ms * 1e-3) / 1e9 / DATASHEET_HBM_GBS,
            **({"traffic": tr["bytes"], "traffic_source": tr["source"]} if T == 32768 else {"traffic": None})}


def measure_prefill_attention(wl, peaks, lengths=(4096, 16384)):
    """kvd_prefill_attention: causal attention of T tokens of one sequence to themselves (a prefill, or the replay of
    an evicted prefix when one residual row per token is kept), one launch of the tcgen05 kernel.  Flops are the causal
    ones, 4 * n_q * d_head per (query, visible key) pair; the peak is the measured bf16 burst figure."""
    import torch
    import paper_2603_19664_b200 as kvd
    shape, kdim = wl.shape, wl.kdim
    out = {"kernel": "kvd_prefill_attn_tc_kernel<256,2> (CTA pairs, tcgen05.mma.cta_group::2, scores and output in tensor memory)",
           "bound": "tensor", "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "cases": []}
    for T in lengths:
        desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                             shape.qk_norm, shape.rms_eps, shape.rope_style, 1, T + 8, 1)
        ctx = kvd.Kvd(desc)
        ctx.kvd_set_layer(0, wl.w_kv, wl.g_in, wl.g_k, shape.rope_theta, 0)
        gen = torch.Generator(device="cuda").manual_seed(7)
        K = torch.randn((T, kdim), device="cuda", generator=gen).to(torch.bfloat16)
        V = torch.randn((T, kdim), device="cuda", generator=gen).to(torch.bfloat16)
        q = torch.randn((T, shape.n_q_heads, shape.d_head), device="cuda", generator=gen).to(torch.bfloat16)
        o = torch.empty_like(q)
        qp = torch.arange(T, dtype=torch.int32, device="cuda")
        for _ in range(3):
            ctx.kvd_prefill_attention(0, T, q, qp, [(K, V, kdim, 0, T)], 0.0, o)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 20
        a.record()
        for _ in range(reps):
            ctx.kvd_prefill_attention(0, T, q, qp, [(K, V, kdim, 0, T)], 0.0, o)
        b.record()
        torch.cuda.synchronize()
        if ctx.kvd_poll_status() != kvd.KVD_OK:
            raise RuntimeError("device status after prefill attention")
        us = a.elapsed_time(b) * 1e3 / reps
        flops = 4.0 * (T * (T + 1) / 2) * shape.n_q_heads * shape.d_head
        out["cases"].append({"tokens": T, "avg_us": us, "achieved": flops / us * 1e-6,
                             "frac": flops / us * 1e-6 / peaks["bf16_tflops"], "causal_gflop": flops * 1e-9})
        ctx.close()
    return out


def run_sweep(wl, peaks):
    """Recompute-vs-read over T (the paper's Section 5.8 measurement, on this hardware)."""
    import torch
    rows = []
    shape, kdim = wl.shape, wl.kdim
    big_T = 32768
    from kvd_synth import make_layer_weights  # noqa: F401
    import paper_2603_19664_b200 as kvd
    desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                         shape.qk_norm, shape.rms_eps, shape.rope_style, 5, big_T + 8, 1)
    ctx = kvd.Kvd(desc)
    ctx.kvd_set_layer(0, wl.w_kv, wl.g_in, wl.g_k, shape.rope_theta, 0)
    ws = torch.empty(kvd.kvd_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_workspace(ws)
    n_sets = 5
    arena = torch.empty(kvd.kvd_store_bytes(desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store(arena, 1)
    X = [torch.randn((big_T, shape.d_hidden), device="cuda", dtype=torch.float32).to(torch.bfloat16) for _ in range(n_sets)]
    K = [torch.randn((big_T + 1, kdim), device="cuda", dtype=torch.float32).to(torch.bfloat16) for _ in range(n_sets)]
    V = [torch.randn((big_T + 1, kdim), device="cuda", dtype=torch.float32).to(torch.bfloat16) for _ in range(n_sets)]
    Ko = torch.empty((big_T, kdim), device="cuda", dtype=torch.bfloat16)
    Vo = torch.empty_like(Ko)
    dst = torch.empty((2, big_T, kdim), device="cuda", dtype=torch.bfloat16)
    pos = torch.arange(big_T, dtype=torch.int32, device="cuda")
    arena8 = torch.empty(kvd.kvd_store_bytes_fp8(desc, 1), dtype=torch.uint8, device="cuda")
    ctx.kvd_attach_store_fp8(arena8, 1)
    for s_ in range(n_sets):  # the rows are recomputed from the store, as the method does (set = sequence slot)
        ctx.kvd_checkpoint_residual(s_, 0, X[s_], pos, big_T)
        ctx.kvd_checkpoint_residual_fp8(s_, 0, X[s_], pos, big_T)
    q = wl.q[:1]
    out = wl.out[:1]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def timed(fn, n=20):
        ts = []
        for i in range(n + 3):
            flush.zero_()  # evict L2 between iterations (the small T cases fit in it)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn(i)
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b))
        return float(np.median(ts))

    side = torch.cuda.Stream()

    def replayed(fn, reps=10):
        """ms per call from a CUDA graph of n_sets back-to-back calls on rotating inputs (no L2 flush:
        below T = 8192 the inputs stay L2-resident, as they are right after being produced)."""
        for i in range(n_sets):
            fn(i)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for i in range(n_sets):
                fn(i)
        g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (reps * n_sets)

    for T in (1, 10, 50, 100, 256, 500, 512, 1024, 2048, 4096, 8192, 16384, 32768):
        def f_rec(i):
            ctx.kvd_recompute_kv(0, None, None, T, Ko, Vo, kdim, seq=i % n_sets, first_row=0)

        def f_att(i):
            ctx.kvd_decode_attention(0, 1, q, [T], [[(K[i % n_sets], V[i % n_sets], kdim, 0, T + 1)]], 0.0, out)

        def f_cp(i):
            dst[0, :T].copy_(K[i % n_sets][:T])
            dst[1, :T].copy_(V[i % n_sets][:T])

        # recompute + attention over the T rebuilt keys: two calls against the fused call, bf16 and FP8 checkpoints
        def f_two(i):
            ctx.kvd_recompute_kv(0, None, None, T, Ko, Vo, kdim, seq=i % n_sets, first_row=0)
            ctx.kvd_decode_attention(0, 1, q, [T], [[(Ko, Vo, kdim, 0, T)]], 0.0, out)

        def f_fused(i):
            ctx.kvd_decode_attention_recompute(0, 1, q, [T], [(i % n_sets, 0, T)], None, None, 0, None, None, kdim,
                                               [[]], 0.0, out)

        def f_rec8(i):
            ctx.kvd_recompute_kv_fp8(0, [(i % n_sets, 0, T, Ko, Vo)], kdim)

        def f_two8(i):
            ctx.kvd_recompute_kv_fp8(0, [(i % n_sets, 0, T, Ko, Vo)], kdim)
            ctx.kvd_decode_attention(0, 1, q, [T], [[(Ko, Vo, kdim, 0, T)]], 0.0, out)

        def f_fused8(i):
            ctx.kvd_decode_attention_recompute_fp8(0, 1, q, [T], [(i % n_sets, 0, T)], [], kdim, [[]], 0.0, out)

        rec, att, cpy = timed(f_rec), timed(f_att), timed(f_cp)
        rec_g, att_g, cpy_g = replayed(f_rec), replayed(f_att), replayed(f_cp)
        variants = {"recompute_fp8_replay_us": replayed(f_rec8) * 1e3,
                    "recompute_then_attention_replay_us": replayed(f_two) * 1e3,
                    "fused_replay_us": replayed(f_fused) * 1e3,
                    "recompute_fp8_then_attention_replay_us": replayed(f_two8) * 1e3,
                    "fused_fp8_replay_us": replayed(f_fused8) * 1e3}
        flops = 4.0 * T * shape.n_kv_heads * shape.d_hidden * shape.d_head
        byts = T * 4 * shape.n_kv_heads * shape.d_head
        rows.append({"T": T,
                     # one eager call after an L2 flush, CUDA events around it (includes launch latency)
                     "recompute_us": rec * 1e3, "attention_us": att * 1e3, "copy_us": cpy * 1e3,
                     "ratio_recompute_over_copy": rec / cpy,
                     # back-to-back graph replays
                     "recompute_replay_us": rec_g * 1e3, "recompute_replay_tflops": flops / (rec_g * 1e-3) / 1e12,
                     "attention_replay_us": att_g * 1e3, "attention_replay_gbs": byts / (att_g * 1e-3) / 1e9,
                     "copy_replay_us": cpy_g * 1e3, "ratio_replay_recompute_over_copy": rec_g / cpy_g,
                     "ratio_replay_recompute_over_attention_read": rec_g / att_g, **variants})
    ctx.close()
    return rows


def run_stack_configs(args):
    """Hot-path timing of the stack-shaped configurations: the 34-layer Gemma-3-4B-shaped stack
    (context 2048, 256 live K/V, batch 1..64: KV-Direct decode step against a full-cache step) and the
    Qwen3-4B-shaped long-context case (36 layers, context 32768, batch 8, 512 live K/V).  Only the
    library's kernels are timed (CUDA graphs of the launch sequence, stored K/V rotating over sets that
    exceed the L2); one layer of each kind is measured and multiplied by the layer count."""
    import torch
    import paper_2603_19664_b200 as kvd
    from kvd_synth import GEMMA3_4B_GLOBAL, GEMMA3_4B_LOCAL, QWEN3_4B, make_layer_weights
    from paper_2603_19664_b200.build import build
    build()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    peaks = load_peaks()

    def dev(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    side = torch.cuda.Stream()

    def timed_graph(fn, n_sets, reps=5):
        """us per call of fn(i), i rotating over n_sets input sets, replayed from a CUDA graph."""
        for i in range(n_sets):
            fn(i)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for i in range(n_sets):
                fn(i)
        g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (reps * n_sets) * 1e3

    def layer_case(shape, ctx_len, budget, batch):
        """One layer, decode step of `batch` sequences at position ctx_len.  KV-Direct: recompute the
        evicted rows of every sequence from the residual store together with K_t, V_t of the new tokens
        (one launch), then attention over recomputed + window + current segments.  Full cache: K_t, V_t,
        then attention over the stored K/V.  Stored K/V rotate over enough sets to exceed the L2."""
        kdim = shape.n_kv_heads * shape.d_head
        lo = 0 if shape.sliding_window == 0 else max(0, ctx_len - shape.sliding_window + 1)
        n_old = max(0, ctx_len - budget - lo)  # evicted positions [lo, ctx_len - budget) this layer attends to
        w = make_layer_weights(shape)
        desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                             shape.qk_norm, shape.rms_eps, shape.rope_style, batch, ctx_len + 8, batch)
        c = kvd.Kvd(desc)
        tw, tg = dev(w.w_kv), dev(w.gamma_in)
        tk = dev(w.gamma_k) if w.gamma_k is not None else None
        c.kvd_set_layer(0, tw, tg, tk, shape.rope_theta, shape.sliding_window)
        ws = torch.empty(kvd.kvd_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
        c.kvd_attach_workspace(ws)
        arena = torch.empty(kvd.kvd_store_bytes(desc, 1), dtype=torch.uint8, device="cuda")
        c.kvd_attach_store(arena, 1)
        xs = torch.randn((ctx_len, shape.d_hidden), device="cuda").to(torch.bfloat16)
        ps = torch.arange(ctx_len, device="cuda", dtype=torch.int32)
        arena8 = torch.empty(kvd.kvd_store_bytes_fp8(desc, 1), dtype=torch.uint8, device="cuda")
        c.kvd_attach_store_fp8(arena8, 1)
        for b in range(batch):
            c.kvd_checkpoint_residual(b, 0, xs, ps, ctx_len)  # STORE_RESIDUAL of the whole context
            c.kvd_checkpoint_residual_fp8(b, 0, xs, ps, ctx_len)  # and as E4M3 checkpoints (second store)
        M = batch * n_old
        Ko = torch.empty((max(M, 1), kdim), device="cuda", dtype=torch.bfloat16)
        Vo = torch.empty_like(Ko)
        set_bytes = 2 * batch * (ctx_len + 1) * kdim * 2
        n_sets = max(2, min(24, -(-300_000_000 // set_bytes)))
        Kf = [torch.randn((batch, ctx_len + 1, kdim), device="cuda").to(torch.bfloat16) for _ in range(n_sets)]
        Vf = [torch.randn((batch, ctx_len + 1, kdim), device="cuda").to(torch.bfloat16) for _ in range(n_sets)]
        xc = torch.randn((batch, shape.d_hidden), device="cuda").to(torch.bfloat16)
        pc = torch.full((batch,), ctx_len, device="cuda", dtype=torch.int32)
        kc = torch.empty((batch, kdim), device="cuda", dtype=torch.bfloat16)
        vc = torch.empty_like(kc)
        q = torch.randn((batch, shape.n_q_heads, shape.d_head), device="cuda").to(torch.bfloat16)
        out = torch.empty_like(q)
        wf = ctx_len - budget
        ranges = [(b, lo, n_old, Ko[b * n_old:], Vo[b * n_old:]) for b in range(batch)] if n_old > 0 else []
        segs_kvd = [[[(Ko[b * n_old:], Vo[b * n_old:], kdim, lo, n_old), (Kf[s][b, wf:], Vf[s][b, wf:], kdim, wf, budget),
                      (kc[b:], vc[b:], kdim, ctx_len, 1)] for b in range(batch)] for s in range(n_sets)]
        segs_full = [[[(Kf[s][b, lo:], Vf[s][b, lo:], kdim, lo, ctx_len + 1 - lo)] for b in range(batch)]
                     for s in range(n_sets)]
        qpos = [ctx_len] * batch

        def rec(i):
            c.kvd_recompute_kv_step(0, ranges, xc, pc, batch, kc, vc, kdim)

        def cur(i):
            c.kvd_recompute_kv(0, xc, pc, batch, kc, vc, kdim)

        def att(i):
            c.kvd_decode_attention(0, batch, q, qpos, segs_kvd[i % n_sets], 0.0, out)

        def att_full(i):
            c.kvd_decode_attention(0, batch, q, qpos, segs_full[i % n_sets], 0.0, out)

        def layer_kvd(i):
            rec(i)
            att(i)

        def layer_full(i):
            cur(i)
            att_full(i)

        # the KV-Direct layer with the recompute fused into attention (recomputed K/V never written):
        # evicted ranges attended inside the recompute kernel, window + current token as live segments
        segs_live = [[[(Kf[s][b, wf:], Vf[s][b, wf:], kdim, wf, budget), (kc[b:], vc[b:], kdim, ctx_len, 1)]
                      for b in range(batch)] for s in range(n_sets)]
        franges = [(b, lo, n_old) for b in range(batch)]

        def layer_fused(i):
            c.kvd_decode_attention_recompute(0, batch, q, qpos, franges, xc, pc, batch, kc, vc, kdim,
                                             segs_live[i % n_sets], 0.0, out)

        # the same two layer forms with the evicted rows taken from the FP8 store.  K_t, V_t of the new tokens
        # come from their quantised rows inside the same launch: up to 8 sequences from the FP8 store (one
        # 256-row block per sequence), larger batches from one contiguous buffer that kvd_quantize_rows_fp8 fills
        # (one block for the whole batch; the small quantising launch is part of the timed layer)
        new_in_store = batch <= 8
        if new_in_store:
            for b in range(batch):
                c.kvd_checkpoint_residual_fp8(b, 0, xc[b:b + 1], pc[b:b + 1], 1)
        new_ranges = [(b, ctx_len, 1, kc[b:], vc[b:]) for b in range(batch)] if new_in_store else []
        codes_c = torch.empty((batch, shape.d_hidden), dtype=torch.uint8, device="cuda")
        scales_c = torch.empty((batch,), dtype=torch.float32, device="cuda")
        sumsq_c = torch.empty_like(scales_c)
        new_rows = None if new_in_store else (codes_c, scales_c, sumsq_c, pc, batch, kc, vc)

        def layer_fp8(i):
            if not new_in_store:
                c.kvd_quantize_rows_fp8(xc, batch, codes_c, scales_c, sumsq_c)
            c.kvd_recompute_kv_fp8_rows(0, ranges + new_ranges, new_rows, kdim)
            att(i)

        def layer_fp8_fused(i):
            if not new_in_store:
                c.kvd_quantize_rows_fp8(xc, batch, codes_c, scales_c, sumsq_c)
            c.kvd_decode_attention_recompute_fp8_rows(0, batch, q, qpos, franges, new_ranges, new_rows, kdim,
                                                      segs_live[i % n_sets], 0.0, out)

        # memory-bound cases first, each after a short pause: a long run of GEMMs at the power cap
        # leaves the clocks low for whatever is measured next
        def rested(fn):
            torch.cuda.synchronize()
            time.sleep(0.3)
            return timed_graph(fn, n_sets)
        rec(0)  # the K/V that the KV-Direct attention reads
        t_cur, t_att, t_full = rested(cur), rested(att), rested(att_full)
        t_layer_full = rested(layer_full)
        t_rec, t_layer_kvd = rested(rec), rested(layer_kvd)
        t_layer_fused = rested(layer_fused)
        t_layer_fp8, t_layer_fp8_fused = rested(layer_fp8), rested(layer_fp8_fused)
        assert c.kvd_poll_status() == kvd.KVD_OK
        flops = 4.0 * (M + batch) * shape.n_kv_heads * shape.d_hidden * shape.d_head
        keys = batch * (ctx_len + 1 - lo)
        byts = keys * 4 * shape.n_kv_heads * shape.d_head
        c.close()
        return {"rows_recomputed": M, "kv_buffer_sets": n_sets,
                "recompute_with_current_us": t_rec, "recompute_tflops": flops / t_rec / 1e6,
                "current_kv_only_us": t_cur, "attention_us": t_att, "attention_gbs": byts / t_att / 1e3,
                "fullcache_attention_us": t_full, "fullcache_attention_gbs": byts / t_full / 1e3,
                "kvdirect_layer_us": t_layer_kvd, "kvdirect_fused_layer_us": t_layer_fused,
                "kvdirect_fp8_layer_us": t_layer_fp8, "kvdirect_fp8_fused_layer_us": t_layer_fp8_fused,
                "fullcache_layer_us": t_layer_full}

    result = {"peaks": peaks, "gemma3_4b_stack_ctx2048_window256": [], "qwen3_4b_ctx32768_batch8_window512": None}
    for batch in (1, 4, 16, 64):
        g = layer_case(GEMMA3_4B_GLOBAL, 2048, 256, batch)
        l = layer_case(GEMMA3_4B_LOCAL, 2048, 256, batch)
        kvd_step = 5 * g["kvdirect_layer_us"] + 29 * l["kvdirect_layer_us"]
        full_step = 5 * g["fullcache_layer_us"] + 29 * l["fullcache_layer_us"]
        result["gemma3_4b_stack_ctx2048_window256"].append(
            {"batch": batch, "kvdirect_decode_step_us": kvd_step,
             "kvdirect_fused_decode_step_us": 5 * g["kvdirect_fused_layer_us"] + 29 * l["kvdirect_fused_layer_us"],
             "kvdirect_fp8_decode_step_us": 5 * g["kvdirect_fp8_layer_us"] + 29 * l["kvdirect_fp8_layer_us"],
             "kvdirect_fp8_fused_decode_step_us": 5 * g["kvdirect_fp8_fused_layer_us"] + 29 * l["kvdirect_fp8_fused_layer_us"],
             "fullcache_decode_step_us": full_step,
             "ratio": kvd_step / full_step, "recomputed_tokens_per_s": batch * (5 * g["rows_recomputed"] // batch +
             29 * l["rows_recomputed"] // batch) / (kvd_step * 1e-6), "global_layer": g, "local_layer": l})
    qw = layer_case(QWEN3_4B, 32768, 512, 8)
    qw["step_us_36_layers"] = 36 * qw["kvdirect_layer_us"]
    qw["fused_step_us_36_layers"] = 36 * qw["kvdirect_fused_layer_us"]
    qw["fp8_step_us_36_layers"] = 36 * qw["kvdirect_fp8_layer_us"]
    qw["fp8_fused_step_us_36_layers"] = 36 * qw["kvdirect_fp8_fused_layer_us"]
    qw["fullcache_step_us_36_layers"] = 36 * qw["fullcache_layer_us"]
    qw["recompute_frac_of_sustained_peak"] = qw["recompute_tflops"] / peaks["bf16_tflops_sustained"]
    qw["recompute_frac_of_burst_peak"] = qw["recompute_tflops"] / peaks["bf16_tflops"]
    qw["attention_frac_of_hbm_peak"] = qw["attention_gbs"] / peaks["hbm_gbs"]
    result["qwen3_4b_ctx32768_batch8_window512"] = qw
    print(json.dumps({"stack_configs": result}), flush=True)


def run_profile_qwen(args):
    """A few eager launches of the Qwen3-4B-shaped layer's kernels for a profiler (a reduced form of
    the long-context configuration: 16384 recomputed rows, decode attention over 2 x 16385 keys in
    recomputed + window + current segments, 268 MB of K and V): no graphs, no measurements."""
    import torch
    import paper_2603_19664_b200 as kvd
    from kvd_synth import QWEN3_4B as shape, make_layer_weights
    from paper_2603_19664_b200.build import build
    build()
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))

    def dev(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    batch, ctx_len, budget = 2, 16384, 512
    kdim = shape.n_kv_heads * shape.d_head
    w = make_layer_weights(shape)
    desc = kvd.make_desc(1, shape.d_hidden, shape.n_q_heads, shape.n_kv_heads, shape.d_head, shape.rms_eps,
                         shape.qk_norm, shape.rms_eps, shape.rope_style, batch, ctx_len + 8, batch)
    c = kvd.Kvd(desc)
    tw, tg, tk = dev(w.w_kv), dev(w.gamma_in), dev(w.gamma_k)
    c.kvd_set_layer(0, tw, tg, tk, shape.rope_theta, 0)
    ws = torch.empty(kvd.kvd_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    c.kvd_attach_workspace(ws)
    arena = torch.empty(kvd.kvd_store_bytes(desc, 1), dtype=torch.uint8, device="cuda")
    c.kvd_attach_store(arena, 1)
    xs = torch.randn((ctx_len, shape.d_hidden), device="cuda").to(torch.bfloat16)
    ps = torch.arange(ctx_len, device="cuda", dtype=torch.int32)
    for b in range(batch):
        c.kvd_checkpoint_residual(b, 0, xs, ps, ctx_len)
    n_old = ctx_len - budget
    Ko = torch.empty((batch * n_old, kdim), device="cuda", dtype=torch.bfloat16)
    Vo = torch.empty_like(Ko)
    n_sets = 3
    Kf = [torch.randn((batch, ctx_len + 1, kdim), device="cuda").to(torch.bfloat16) for _ in range(n_sets)]
    Vf = [torch.randn((batch, ctx_len + 1, kdim), device="cuda").to(torch.bfloat16) for _ in range(n_sets)]
    xc = torch.randn((batch, shape.d_hidden), device="cuda").to(torch.bfloat16)
    pc = torch.full((batch,), ctx_len, device="cuda", dtype=torch.int32)
    kc = torch.empty((batch, kdim), device="cuda", dtype=torch.bfloat16)
    vc = torch.empty_like(kc)
    q = torch.randn((batch, shape.n_q_heads, shape.d_head), device="cuda").to(torch.bfloat16)
    out = torch.empty_like(q)
    ranges = [(b, 0, n_old, Ko[b * n_old:], Vo[b * n_old:]) for b in range(batch)]
    for i in range(max(args.steps, 1) + 2):
        s = i % n_sets
        c.kvd_recompute_kv_step(0, ranges, xc, pc, batch, kc, vc, kdim)
        segs = [[(Ko[b * n_old:], Vo[b * n_old:], kdim, 0, n_old),
                 (Kf[s][b, n_old:], Vf[s][b, n_old:], kdim, n_old, budget), (kc[b:], vc[b:], kdim, ctx_len, 1)]
                for b in range(batch)]
        c.kvd_decode_attention(0, batch, q, [ctx_len] * batch, segs, 0.0, out)
        # the same keys from one stored segment (the cached-KV read)
        c.kvd_decode_attention(0, batch, q, [ctx_len] * batch,
                               [[(Kf[s][b], Vf[s][b], kdim, 0, ctx_len + 1)] for b in range(batch)], 0.0, out)
        # the KV-Direct layer again with the recompute fused into attention (every second launch of the
        # recompute kernel in this run is the fused variant)
        c.kvd_decode_attention_recompute(0, batch, q, [ctx_len] * batch, [(b, 0, n_old) for b in range(batch)], xc, pc,
                                         batch, kc, vc, kdim,
                                         [[(Kf[s][b, n_old:], Vf[s][b, n_old:], kdim, n_old, budget),
                                           (kc[b:], vc[b:], kdim, ctx_len, 1)] for b in range(batch)], 0.0, out)
    torch.cuda.synchronize()
    assert c.kvd_poll_status() == kvd.KVD_OK
    print(json.dumps({"profile_run": "qwen3-4b layer", "rows_recomputed": batch * n_old, "keys": batch * (ctx_len + 1),
                      "launches": c.kvd_launch_count()}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="kvd", choices=["kvd", "reference"])
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--sets", type=int, default=N_SETS, help="rotating buffer sets (each ~59 MB)")
    ap.add_argument("--profile", action="store_true", help="eager launches only, for a run under a profiler")
    ap.add_argument("--profile-prefill-attn", action="store_true",
                    help="with --profile: also launch kvd_prefill_attention over 4096 tokens a few times")
    ap.add_argument("--profile-long-attn", action="store_true",
                    help="with --profile: also run decode attention over 32769 keys a few times")
    ap.add_argument("--profile-qwen", action="store_true",
                    help="eager launches of the Qwen3-4B-shaped layer's kernels (reduced long-context case) for a profiler")
    ap.add_argument("--profile-stack", action="store_true",
                    help="eager launches of whole-stack decode steps (batch 4) for a run under a profiler")
    ap.add_argument("--no-stack", action="store_true", help="skip the whole-stack decode step (configs 3 and 5)")
    ap.add_argument("--short-session", action="store_true", help="config 5 with 3 turns of 16 tokens instead of 20 of 128")
    ap.add_argument("--stack-all", action="store_true", help="whole-stack decode step at batch 1, 4, 16 and 64")
    ap.add_argument("--stack-configs", action="store_true",
                    help="time the hot path of the stack-shaped configurations instead of the contract line")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.profile_qwen:
        run_profile_qwen(args)
    elif args.profile_stack:
        run_profile_stack(args)
    elif args.stack_configs:
        run_stack_configs(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
