#!/usr/bin/env python
"""Benchmark of the SPLA decode step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One *step* = one pass of the whole hot path over one batch of synthetic input: append one token per
sequence (cache write, block statistics, recurrent state) and decode (block score, top-k, sparse attention,
residual linear attention, merge).  Metric: decode-attention queries x heads per second (batch * H_q per step),
whole job, at the 128K-context configuration, plus the HBM roofline of the dominant kernel.

Timing: W warm-up steps, then exactly K steps between barrier + synchronize, timed with CUDA events on the
launching stream, max over ranks.  The steps rotate over R independent caches so that the bytes touched per
rotation exceed three times the L2 size (cold-L2 protocol).  Steps are replayed from a CUDA graph of min(K, 64)
steps (plus one of the remainder) so that the Python launch path is not what is measured.  One JSON line is printed
by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attention_query_heads_per_s"
UNIT = "query_heads/s"
L2_BYTES = 126 * 1024 * 1024
GRAPH_STEPS = 64
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from ncu captures of this command
# on a small case (one cache, a few launches), per workload
NCU_TRAFFIC = {"long_128k": 106.4e6, "long_128k+windows(C=32,s=16)": 241.2e6, "long_128k+stats_bf16": 70.4e6, "gqa_32k": 72.6e6, "very_long_1m": 86.2e6,
               "long_128k+n_q_heads=40": 108.2e6}


# ------------------------------------------------------------------------------------------------------------
# CPU baseline: the float64 oracle, as it stands, on the host cores (also the --impl reference arm)
# ------------------------------------------------------------------------------------------------------------
_ORACLE_UNITS = None
WINDOW = None          # (C, s) when --window is given: strided selection windows instead of whole blocks
STATS_BF16 = False     # --stats-bf16: the block statistics are stored (and streamed) as bfloat16


def _oracle_worker(args):
    """Times incremental-form oracle decodes of one unit (block statistics and state cached, as a server would)."""
    idx, n_dec, cfg = args
    from threadpoolctl import threadpool_limits
    from oracle import spla_oracle as O
    K, V, qs, gam = _ORACLE_UNITS[idx]
    with threadpool_limits(limits=1):
        cache = O.UnitCache.from_prefill(K, V, cfg["block_size"], window=cfg["window"])
        t0 = time.perf_counter()
        for i in range(n_dec):
            cache.decode(qs[i % len(qs)], gam, top_k=cfg["top_k"], n_sink=cfg["n_sink"], n_local=cfg["n_local"],
                         stats_bf16=cfg["stats_bf16"])
        return time.perf_counter() - t0


def oracle_throughput(w, n_dec_per_unit: int, repeats: int = 1, max_units: int = 0):
    """Runs the oracle on one sequence's KV heads (one unit per process; at most `max_units` processes when given).
    Returns (query_heads/s list, cores, sample)."""
    global _ORACLE_UNITS
    import multiprocessing as mp
    import numpy as np
    from paper_2601_22379_b200 import synth
    cores = len(os.sched_getaffinity(0))
    n_units = max(1, min(cores, w.n_kv_heads))
    if max_units > 0:
        n_units = min(n_units, max_units)
    K, V = synth.prefill_kv(w, 0, "cpu")
    G = w.group
    gam = synth.gamma(w).double().numpy()
    qs = [synth.step_queries(w, s, "cpu")[0].double().numpy() for s in range(8)]
    _ORACLE_UNITS = [(K[h].double().numpy(), V[h].double().numpy(), [q[h * G:(h + 1) * G] for q in qs],
                      gam[h * G:(h + 1) * G]) for h in range(n_units)]
    del K, V
    cfg = dict(block_size=w.block_size, top_k=w.top_k, n_sink=w.n_sink, n_local=w.n_local, window=WINDOW,
               stats_bf16=STATS_BF16)
    values = []
    ctx = mp.get_context("fork")
    with ctx.Pool(n_units) as pool:
        for _ in range(repeats):
            times = pool.map(_oracle_worker, [(i, n_dec_per_unit, cfg) for i in range(n_units)])
            values.append(n_units * n_dec_per_unit * G / max(times))
    _ORACLE_UNITS = None
    sample = (f"{n_units} units (sequence 0, KV heads 0..{n_units - 1}) of {workload_name(w)}, {n_dec_per_unit} decode calls each, "
              f"float64 numpy oracle with cached block statistics and state, one process per unit")
    return values, n_units, sample


def run_reference(args, w):
    """--impl reference: the oracle timed on the host cores, same metric and config."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = args.steps, max(args.warmup, 0)
    n_dec = 200
    t0 = time.perf_counter()
    vals, cores, sample = oracle_throughput(w, n_dec, repeats=max(1, min(steps + warmup, 6)))
    vals = vals[min(warmup, len(vals) - 1):] or vals
    value = statistics.mean(vals)
    line = base_line(args, w, value, ms_per_step=1e3 * w.batch * w.n_q_heads / value)
    line.update({"impl": "reference", "dtype": "f64", "n_gpus": args.gpus,
                 "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
                 "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                 "gpu_launches": 0, "wall_s": time.perf_counter() - t0})
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------------------
def n_windows(w):
    return (w.block_size - WINDOW[0]) // WINDOW[1] + 1 if WINDOW else 1


def workload_name(w):
    from paper_2601_22379_b200 import synth
    base = synth.BY_NAME[w.name]
    over = "".join(f"+{k}={getattr(w, k)}" for k in ("batch", "context", "n_q_heads") if getattr(w, k) != getattr(base, k))
    return w.name + over + (f"+windows(C={WINDOW[0]},s={WINDOW[1]})" if WINDOW else "") + ("+stats_bf16" if STATS_BF16 else "")


def stat_bytes():
    return 2 if STATS_BF16 else 4


def base_line(args, w, value, ms_per_step):
    from paper_2601_22379_b200 import synth
    by = synth.algorithmic_bytes_per_step(w, n_windows=n_windows(w), stat_bytes=stat_bytes())
    return {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w.kv_dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": workload_name(w), "batch": w.batch, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
                   "head_dim": w.head_dim, "context": w.context, "block_size": w.block_size, "top_k": w.top_k,
                   "n_sink": w.n_sink, "n_local": w.n_local, "kv_dtype": w.kv_dtype,
                   "selection": (f"strided windows C={WINDOW[0]} s={WINDOW[1]}, max-pooled per block" if WINDOW
                                 else "whole-block statistics") + (", statistics stored as bfloat16" if STATS_BF16 else ""),
                   "algorithmic_bytes_per_step": by["total"], "dense_kv_bytes_per_step": by["dense_kv"],
                   "parallelism": f"replicas x{args.gpus} (units are independent; no collective)"},
    }


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        rows = [r for t, r in self.rows if t0 <= t <= t1] or [r for _, r in self.rows[-3:]]
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def run_ours(args, w):
    import torch
    from paper_2601_22379_b200 import binding, build, replicas, runner, synth

    world, rank, local = replicas.env_world()
    cpu_base = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        vals, cores, sample = oracle_throughput(w, 400, repeats=2)      # before CUDA is initialised (fork)
        one, _, sample1 = oracle_throughput(w, 300, repeats=1, max_units=1)
        cpu_base = {"value": vals[-1], "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                    "single_thread": {"value": one[-1], "unit": UNIT, "cores": 1, "sample": sample1}}

    build.build()
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    replicas.init("nccl", dev)

    steps, warmup = args.steps, max(args.warmup, 3)
    by = synth.algorithmic_bytes_per_step(w, n_windows=n_windows(w), stat_bytes=stat_bytes())
    R = 2                                                             # caches to rotate over (cold-L2 protocol)
    while R * by["total"] < 3 * L2_BYTES and R < GRAPH_STEPS:
        R *= 2
    if args.caches > 0:                                               # profiling aid: fewer caches, less device memory
        R = args.caches
    n_e2e = max(8, min(steps, 256))
    G1 = max(1, min(steps, GRAPH_STEPS))                              # steps per captured graph
    per_cache = -(-(steps + warmup + 3 * GRAPH_STEPS + n_e2e) // R) + 2 * GRAPH_STEPS
    wl = w.scaled(n_steps=per_cache)
    prefill = runner.generate_prefill(wl, dev)
    caches = []
    for _ in range(R):
        c, _, _, _ = runner.build_cache(wl, dev, prefill=prefill, window=WINDOW,
                                        flags=binding.SPLA_STATS_BF16 if STATS_BF16 else 0)
        caches.append(c)
    del prefill
    n_app = [0] * R                                                   # tokens appended per cache so far

    def set_bounds(exact: bool):
        # The library sizes its grids from a host-side bound of the sequence lengths.  Graph replays append
        # without the host seeing it, so the bound is raised to the capacity while graphs run and put back after.
        for ci, c in enumerate(caches):
            c.set_length_bound(w.context + n_app[ci] if exact else wl.max_context - GRAPH_STEPS)
    gamma = synth.gamma(w).to(dev)
    n_in = GRAPH_STEPS
    qs = [synth.step_queries(w, s, dev) for s in range(n_in)]
    kvs = [synth.step_kv(w, s, dev) for s in range(n_in)]
    outs = [torch.empty(w.batch, w.n_q_heads, w.head_dim, dtype=torch.float32, device=dev) for _ in range(R)]
    stream = torch.cuda.Stream(device=dev)

    def one_step(i):
        c = caches[i % R]
        k1, v1 = kvs[i % n_in]
        c.append_decode(k1, v1, qs[i % n_in], gamma, out=outs[i % R])    # the step: append, then decode, one call

    def decode_only(i):
        caches[i % R].decode(qs[i % n_in], gamma, out=outs[i % R])

    def capture(body, n):
        """A CUDA graph of body(0) .. body(n - 1), replayed once untimed; None for n == 0."""
        if n <= 0:
            return None
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(n):
                body(i)
        g.replay()
        return g

    def appended_by(n):                                               # tokens a graph of n steps appends to each cache
        return [len(range(ci, n, R)) for ci in range(R)]

    n_rep, n_rem = steps // G1, steps % G1
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for i in range(warmup):                                        # eager warm-up steps (also load the kernels)
            one_step(i)
            n_app[i % R] += 1
        set_bounds(exact=False)
        n_launch0 = binding.launch_count()
        graph = capture(one_step, G1)                                  # (the library counts the kernels it records)
        launches_per_step = (binding.launch_count() - n_launch0) / G1
        set_bounds(exact=False)
        graph_rem = capture(one_step, n_rem)
        for n in (G1, n_rem):
            for ci, a in enumerate(appended_by(n)):
                n_app[ci] += a
        n_launch0 = binding.launch_count()
        graph_dec = capture(decode_only, G1)
        launches_per_decode = (binding.launch_count() - n_launch0) / G1
    torch.cuda.synchronize()

    def barrier():
        replicas.barrier(dev)

    # ---- the timed region: exactly `steps` steps ----------------------------------------------------------
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.15)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0 = time.perf_counter()
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(n_rep):
            graph.replay()
        if graph_rem is not None:
            graph_rem.replay()
        e1.record(stream)
    barrier()
    t1 = time.perf_counter()
    total_ms = e0.elapsed_time(e1)
    clocks = sampler.stop(t0, t1)
    for ci, a in enumerate(appended_by(G1)):
        n_app[ci] += n_rep * a
    for ci, a in enumerate(appended_by(n_rem)):
        n_app[ci] += a
    for c in caches:
        st = c.sync_status()
        if st != 0:
            raise RuntimeError(f"device status {st} after the timed region")

    # ---- decode-only (no append) for context, same rotation ---------------------------------------------------
    with torch.cuda.stream(stream):
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_dec_rep = max(1, min(steps // G1, 64))
        d0.record(stream)
        for r in range(n_dec_rep):
            graph_dec.replay()
        d1.record(stream)
    torch.cuda.synchronize()
    dec_ms = d0.elapsed_time(d1) / (n_dec_rep * G1)

    # ---- duration of the dominant kernel (block score + selection): a CUDA graph of back-to-back launches of that
    # kernel alone, rotating over the caches (cold L2), timed with CUDA events on the launching stream -------------
    sel_bufs = [c.new_sel_buffer() for c in caches]
    with torch.cuda.stream(stream):
        for i in range(R):
            caches[i].select(qs[i], sel_bufs[i])                      # warm-up, also loads the kernel
        graph_sel = capture(lambda i: caches[i % R].select(qs[i % n_in], sel_bufs[i % R]), G1)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_sel_rep = max(1, min(steps // G1, 64))
        s0.record(stream)
        for r in range(n_sel_rep):
            graph_sel.replay()
        s1.record(stream)
    torch.cuda.synchronize()
    sc = s0.elapsed_time(s1) / (n_sel_rep * G1)

    # ---- end to end through the public call with host buffers -----------------------------------------------------
    # Per step: the host writes q, k_t, v_t into a pinned staging buffer; the H2D copy, append and decode are enqueued
    # as one captured graph per cache, the output goes device -> host by the merge kernel's own stores into a pinned
    # host buffer (no separate copy), and the stream is synchronised, because the caller reads the output before it
    # can form the next query.  q, k_t and v_t travel in one staging buffer: one host write and one H2D copy per step.
    nq, nk = qs[0].numel(), kvs[0][0].numel()
    src = [torch.cat([qs[i].reshape(-1), kvs[i][0].reshape(-1), kvs[i][1].reshape(-1)]).cpu() for i in range(8)]
    hstage = src[0].clone().pin_memory()
    dstage = torch.empty_like(src[0], device=dev)
    dq = dstage[:nq].view_as(qs[0])
    dk, dv = dstage[nq:nq + nk].view_as(kvs[0][0]), dstage[nq + nk:].view_as(kvs[0][1])
    hout = torch.empty(w.batch, w.n_q_heads, w.head_dim, dtype=torch.float32).pin_memory()
    h2d = hstage.numel() * hstage.element_size()
    d2h = hout.numel() * 4

    def e2e_body(ci):
        dstage.copy_(hstage, non_blocking=True)
        caches[ci].append_decode(dk, dv, dq, gamma, out=hout)   # the merge kernel stores the output straight into pinned host memory

    e2e_graphs = []
    set_bounds(exact=False)
    with torch.cuda.stream(stream):
        for ci in range(R):
            gph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gph, stream=stream):
                e2e_body(ci)
            e2e_graphs.append(gph)
    barrier()
    with torch.cuda.stream(stream):
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for i in range(n_e2e):
            hstage.copy_(src[i % 8])                                   # the step's inputs arrive in host memory
            e2e_graphs[i % R].replay()
            n_app[i % R] += 1
            stream.synchronize()                                       # the caller reads the result before the next step
        g1.record(stream)
    barrier()
    e2e_ms = g0.elapsed_time(g1) / n_e2e
    set_bounds(exact=True)
    for c in caches:
        st = c.sync_status()
        if st != 0:
            raise RuntimeError(f"device status {st} after the end-to-end leg")

    total_ms, e2e_ms = replicas.max_over_ranks([total_ms, e2e_ms], dev)
    value = replicas.whole_job_rate(w.batch * w.n_q_heads, steps, total_ms)

    peak, peak_kind = measured_peaks()
    # The dominant kernel: where one kernel does the whole decode (score + select + attend + merge of every unit) it is
    # that kernel, timed as the decode-only launches above, on all the bytes a decode step must touch; where the decode
    # is two launches, the score + select kernel on the statistics and the state, timed alone.
    fused = launches_per_decode < 1.5
    if fused:
        roof_kernel, roof_bytes, roof_ms = "decode_fused_kernel (score + top-k + attend + merge)", by["total"], dec_ms
    else:
        roof_kernel, roof_bytes, roof_ms = "score_cluster_kernel (block score + top-k)", by["stats"] + by["state"], sc
    achieved = roof_bytes / (roof_ms * 1e-3) / 1e9
    line = base_line(args, w, value, ms_per_step=total_ms / steps)
    line["warmup"] = warmup
    line["config"].update({"l2_protocol": f"rotation over {R} independent caches ({R * by['total'] / 2**20:.0f} MiB per "
                                          f"rotation, > 3x L2) - cold L2", "context_growth_tokens_per_cache": per_cache,
                           "launch": f"CUDA graph of {G1} steps, replayed {n_rep}x" +
                                     (f", plus one of {n_rem} steps" if n_rem else "")})
    line.update({
        "clocks": clocks,
        "e2e": {"value": w.batch * w.n_q_heads * world / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
        "gpu_launches": int(round(launches_per_step * steps)),
        "roofline": {"bound": "hbm", "kernel": roof_kernel, "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "bytes_per_launch": roof_bytes, "ms_per_launch": roof_ms,
                     "traffic": args.traffic if args.traffic is not None else NCU_TRAFFIC.get(workload_name(w))},
        "kernels": {"launches_per_decode": launches_per_decode, "score_select_ms": sc, "decode_minus_score_ms": dec_ms - sc,
                    "decode_only_ms": dec_ms, "decode_only_GBps": by["total"] / (dec_ms * 1e-3) / 1e9,
                    "decode_only_frac_of_peak": by["total"] / (dec_ms * 1e-3) / 1e9 / peak,
                    "decode_only_frac_of_8TBps": by["total"] / (dec_ms * 1e-3) / 8e12,
                    "decode_only_query_heads_per_s": w.batch * w.n_q_heads / (dec_ms * 1e-3)},
    })
    if cpu_base is not None:
        line["cpu_baseline"] = cpu_base
    if rank == 0:
        print(json.dumps(line), flush=True)
    replicas.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8192)
    ap.add_argument("--warmup", type=int, default=64)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long_128k")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--caches", type=int, default=0, help="rotate over this many caches instead of the cold-L2 count "
                    "(for profiler captures, which must hold little device memory)")
    ap.add_argument("--traffic", type=float, default=None,
                    help="DRAM bytes per launch of the dominant kernel from an ncu capture; default: the figure "
                         "recorded in this file for the workload")
    ap.add_argument("--q-heads", type=int, default=0, help="override the number of query heads (the group size is "
                    "q_heads / 8 KV heads; the paper's own model has 40)")
    ap.add_argument("--window", default=None, metavar="C,s",
                    help="strided selection windows (the paper's setting is 32,16) instead of whole-block statistics")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (scaling studies; the metric is quoted on the default)")
    ap.add_argument("--context", type=int, default=0, help="override the workload's context length (scaling studies)")
    ap.add_argument("--stats-bf16", action="store_true",
                    help="store the block statistics as bfloat16 (half the bytes for the score kernel to stream)")
    args = ap.parse_args()
    global WINDOW, STATS_BF16
    if args.window:
        WINDOW = tuple(int(x) for x in args.window.split(","))
    STATS_BF16 = args.stats_bf16
    from paper_2601_22379_b200 import synth
    w = synth.BY_NAME[args.workload]
    if args.batch > 0:
        w = w.scaled(batch=args.batch)
    if args.q_heads > 0:
        w = w.scaled(n_q_heads=args.q_heads)
    if args.context > 0:
        w = w.scaled(context=args.context, context_min=min(w.context_min, args.context))
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
