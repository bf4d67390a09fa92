"""Times the bulk append (prefill) of a workload: cache write, block statistics, recurrent state, lengths.

    python bench_prefill.py [--workload long_128k] [--batch N] [--reps R] [--general]

One JSON line: milliseconds per append of the whole context (CUDA events on the launching stream, after a
warm-up call, each repetition into a fresh cache so that every token is new), tokens/s, and the K/V bytes the
state kernel has to read over the time of the whole append.  `--general` forces the FMA state kernel.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2601_22379_b200 import binding, build, runner, synth  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="long_128k")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (smaller device footprint)")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--general", action="store_true", help="general kernels: the state update runs on the FMA pipe")
    args = ap.parse_args()
    build.build()
    dev = "cuda:0"
    w = synth.BY_NAME[args.workload]
    if args.batch > 0:
        w = w.scaled(batch=args.batch)
    flags = binding.SPLA_GENERAL_KERNELS if args.general else 0
    K, V, lens = runner.generate_prefill(w, dev)
    ragged = bool((lens != K.shape[2]).any().item())
    times = []
    for rep in range(args.reps + 1):
        cache = binding.SplaCache(runner.config_for(w, flags=flags), dev)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cache.append_tokens(K, V, lens if ragged else None)
        e1.record()
        torch.cuda.synchronize()
        assert cache.sync_status() == 0
        if rep > 0:                                   # the first call warms up
            times.append(e0.elapsed_time(e1))
        del cache
    ms = statistics.median(times)
    tokens = int(lens.sum().item())
    kv_bytes = 2 * tokens * w.n_kv_heads * w.head_dim * K.element_size()
    print(json.dumps({
        "workload": w.name, "batch": w.batch, "tokens": tokens, "kernels": "general (FMA state)" if args.general else "default",
        "append_ms": ms, "tokens_per_s": tokens / (ms * 1e-3), "kv_bytes": kv_bytes,
        "kv_read_GBps_over_whole_append": kv_bytes / (ms * 1e-3) / 1e9, "reps": args.reps}))


if __name__ == "__main__":
    main()
