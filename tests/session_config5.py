"""Multi-turn session on a decoder stack (the synthetic restatement of the paper's Section 5.5
experiment): turns alternate a user segment of random token ids with greedily decoded tokens; the
bounded-window policy with recomputation must reproduce the full-cache tokens exactly, and the live
K/V memory stays bounded by the window.

Run directly for the full-size case (34-layer Gemma-3-4B-shaped stack, 20 turns, user segments of
256..1024 tokens, 128 decoded tokens per turn, window 256):
    python tests/session_config5.py [--turns 20] [--gen 128] [--window 256] [--small]
Prints one JSON line per turn and a summary line.

--chained runs the single-checkpoint variant instead (one residual row per token, the evicted
prefix carried through all layers every step: quadratic work, so use short segments, e.g.
    python tests/session_config5.py --chained --turns 3 --gen 8 --window 32 --seg 48 96).
"""
import argparse
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import numpy as np  # noqa: E402
import torch  # noqa: E402

from kvd_synth import GEMMA3_4B_STACK, S_GEMMA, SEED_TOKENS  # noqa: E402
from stack_harness import GpuStack, GpuStackChained, torch_stack_weights  # noqa: E402


def run_session(stack, weights, turns, gen, window, seg_lo, seg_hi, max_tokens, device_weights=True, log=None,
                chained=False, tiled=False):
    """Returns (per-turn records, all-match flag)."""
    rng = np.random.Generator(np.random.PCG64(SEED_TOKENS + 77))
    segments = [rng.integers(0, stack.vocab, size=int(rng.integers(seg_lo, seg_hi + 1))).tolist() for _ in range(turns)]
    if chained:
        full = GpuStack(stack, weights, "full", 0, max_tokens, device_weights, tiled_attention=tiled)
        kvdir = GpuStackChained(stack, weights, window, max_tokens, device_weights, tiled_attention=tiled)
    else:
        full = GpuStack(stack, weights, "full", 0, max_tokens, device_weights, tiled_attention=tiled)
        kvdir = GpuStack(stack, weights, "kvdirect", window, max_tokens, device_weights, tiled_attention=tiled)
    records, all_match = [], True
    for t in range(turns):
        outs = []
        for m in (full, kvdir):
            t0 = time.perf_counter()
            logits = m.prefill(segments[t])
            toks = []
            for _ in range(gen):
                nxt = m.greedy_token()
                toks.append(nxt)
                logits = m.step(nxt)
            torch.cuda.synchronize()
            outs.append((toks, time.perf_counter() - t0))
        match = outs[0][0] == outs[1][0]
        all_match &= match
        rep_f, rep_k = full.memory_report(), kvdir.memory_report()
        rec = {"turn": t + 1, "tokens_so_far": kvdir.t, "user_tokens": len(segments[t]), "generated": gen,
               "token_match": match, "seconds_full_cache": outs[0][1], "seconds_kvdirect": outs[1][1],
               "full_cache_kv_bytes": rep_f["live_kv_bytes"], "kvdirect_live_kv_bytes": rep_k["live_kv_bytes"],
               "kvdirect_checkpoint_bytes_per_layer_rows": rep_k.get("checkpoint_bytes_per_layer_rows"),
               "kvdirect_checkpoint_bytes_single_row": rep_k.get("checkpoint_bytes_single_row"),
               "rows_replayed_so_far": getattr(kvdir, "replayed_rows", 0),
               "kvdirect_eq28_bytes_single_checkpoint_accounting": rep_k["eq28_bytes"],
               "rows_recomputed_so_far": kvdir.recomputed_rows}
        records.append(rec)
        if log:
            log(json.dumps(rec))
    return records, all_match


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--turns", type=int, default=20)
    ap.add_argument("--gen", type=int, default=128)
    ap.add_argument("--window", type=int, default=256)
    ap.add_argument("--small", action="store_true", help="small 6-layer stack instead of the 34-layer one")
    ap.add_argument("--chained", action="store_true", help="one checkpointed row per token, chained recompute")
    ap.add_argument("--seg", type=int, nargs=2, default=None, help="user segment length range")
    ap.add_argument("--tiled", action="store_true", help="all attention through kvd_prefill_attention (row-tiled kernel)")
    a = ap.parse_args()
    stack = S_GEMMA if a.small else GEMMA3_4B_STACK
    seg = tuple(a.seg) if a.seg else ((24, 64) if a.small else (256, 1024))
    max_tokens = a.turns * (seg[1] + a.gen) + 8
    w = torch_stack_weights(stack)
    recs, ok = run_session(stack, w, a.turns, a.gen, a.window, seg[0], seg[1], max_tokens,
                           log=lambda s: print(s, flush=True), chained=a.chained, tiled=a.tiled)
    print(json.dumps({"summary": True, "stack": stack.name, "turns": a.turns, "all_tokens_match": ok,
                      "peak_full_cache_kv_bytes": max(r["full_cache_kv_bytes"] for r in recs),
                      "peak_kvdirect_live_kv_bytes": max(r["kvdirect_live_kv_bytes"] for r in recs),
                      "final_checkpoint_bytes": recs[-1]["kvdirect_checkpoint_bytes_single_row"] if a.chained
                      else recs[-1]["kvdirect_checkpoint_bytes_per_layer_rows"],
                      "eq28_bytes": recs[-1]["kvdirect_eq28_bytes_single_checkpoint_accounting"]}), flush=True)
    sys.exit(0 if ok else 1)


if __name__ == "__main__":
    main()
