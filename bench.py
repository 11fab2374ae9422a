#!/usr/bin/env python
"""Benchmark of the ChunkWise-LoRA hot path on B200.

Headline workload (default): the 32-layer LLaMA-7B-shaped projection stack, 4 sequences x 4096 tokens.  One step =
one pass of the whole hot path over that batch: per layer, token scoring from fp32 logits [16384, 32000], adaptive
partition and rank selection, then the adapted projection for all seven projections (q, k, v, o, gate, up, down)
with R = 64.  Prints ONE JSON line: metric, value (whole-job tokens/s), ms_per_step, config, clocks, e2e (host
buffers in and out every step), gpu_launches, roofline (dominant kernel against the measured peaks), cpu_baseline
(the fp64 oracle timed on the host cores) and, at one GPU, a `configs` block with the same measurement on the other
workloads (single-sequence prefill, packed ragged prefill, decode with a fixed table, decode through the scheduler).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg5|cfg2|cfg3|cfg4|cfg4_stream|cfg1] [--layers L] [--min-seconds S]
                    [--no-configs] [--no-group] [--decode-mode batch|lanes|serial] [--prefetch-mb M] [--lean]

Every timed region lasts at least --min-seconds of device time: the block of K steps is repeated (`inner_repeats`)
until it does, and ms_per_step is the mean over all K x repeats steps (median and min per block are beside it).

N > 1 runs N independent replicas (one process per GPU; without a launcher the script starts its own ranks through
torch.distributed.run); the path has no exchange step, so there is no data-path collective: only the timing barrier
and the max-over-ranks reduction of the timed region.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "adapted_projection_tokens_per_s"
UNIT = "tokens/s"
SUB_CONFIGS = ("cfg2", "cfg3", "cfg4", "cfg4_stream")
DECODE_WEIGHT_SETS = 4      # decode steps rotate over this many weight sets so that no step finds its weights in L2


# ------------------------------------------------------------------------------------ helpers
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# Revision tag of the dominant kernel the ncu counters under profiles/ were taken on.  Bump it whenever
# cwl_apply's kernel changes: a traffic figure taken on another revision is reported as null.
APPLY_KERNEL_REVISION = "pairs-256x512-grouped-r11"


def load_traffic(key: str):
    """DRAM bytes per step of the dominant kernel from the committed ncu summary, or None when there is
    no figure for this workload or the kernel has changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    with open(path) as fh:
        for line in fh:
            parts = line.split()
            if len(parts) >= 3 and not line.startswith("#") and parts[0] == key and parts[2] == APPLY_KERNEL_REVISION:
                return float(parts[1])
    return None


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        inside = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.1] or [l for (_, l) in self.lines]
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in inside:
            parts = [x.strip() for x in l.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def table_flops(table: dict, window: int, T: int, projs, R: int):
    """Algorithmic and executed FLOPs of the adapted projections for one step."""
    off, rank, flags = table["offsets"], table["rank"], table["flags"]
    active = np.zeros(T, dtype=np.int64)
    for c in range(table["n_chunks"]):
        active[off[c]:off[c + 1]] = rank[c]
        if c > 0 and not (flags[c] & 1):
            w = min(window, off[c + 1] - off[c])
            active[off[c]:off[c] + w] = max(rank[c], rank[c - 1])
    rsum = int(active.sum())
    alg = sum(2 * T * d_in * d_out + 2 * rsum * (d_in + d_out) for (d_in, d_out) in projs)
    exe = sum(2 * T * d_in * d_out + 2 * T * R * (d_in + d_out) for (d_in, d_out) in projs)
    return alg, exe


def make_workload(name: str):
    from paper_2601_21109_b200 import workloads as wl
    if name == "cfg2":
        return wl.config2()
    if name == "cfg1":
        return wl.config1()
    if name in ("cfg4", "cfg4_stream"):
        w = wl.config4()
        if name == "cfg4_stream":
            # decode through the token-by-token scheduler: per-sequence scores U[0,1) stand in for the scorer's output
            from paper_2601_21109_b200.workloads import Policy
            w.name = "cfg4_decode_streaming_scheduler"
            w.policy = Policy.ladder([8, 16, 32, 64], 32.0, [0.25, 0.5, 0.75], min_len=16, window=8)
            w.score = np.random.default_rng(wl.SEED_BASE + 4).uniform(0, 1, w.T).astype(np.float32)
        return w
    if name == "cfg3":
        return wl.config3()
    if name == "cfg5":
        return wl.config5_layer()
    raise SystemExit(f"unknown workload {name}")


def layers_of(name: str, args) -> int:
    """Weight sets resident on the device: the stack's layers, or the sets a decode run rotates over."""
    if name == "cfg5":
        return args.layers
    return args.weight_sets if name in ("cfg4", "cfg4_stream") else 1


def config_dict(name: str, w, n_layers: int, world: int, grouped: bool) -> dict:
    """What was run, from the workload alone (the same for both arms)."""
    decode = name in ("cfg4", "cfg4_stream")
    streaming = name == "cfg4_stream"
    has_logits, fixed = w.logits is not None, w.table is not None
    parts = (["scheduler step"] if streaming else []) + (["score"] if has_logits else []) + \
        ([] if (fixed or streaming) else ["partition"]) + [f"{len(w.projections)} adapted projections"]
    stack = n_layers if name == "cfg5" else 1
    steps_include = (f"{stack} layers x (" if stack > 1 else "(") + " + ".join(parts) + ")"
    step_bytes = stack * (sum(2 * p.d_in * p.d_out for p in w.projections) +
                          (int(w.logits.size) * 4 if has_logits else 0))
    if decode:
        l2 = (f"steps rotate over {n_layers} distinct weight sets ({n_layers * step_bytes / 1e6:.0f} MB), so every "
              f"step streams its {step_bytes / 1e6:.0f} MB of weights from HBM; no flush needed")
    elif step_bytes > 126e6:
        l2 = f"inputs larger than L2 ({step_bytes / 1e6:.0f} MB of weights and logits read per step); no flush needed"
    else:
        l2 = (f"inputs smaller than L2 ({step_bytes / 1e6:.1f} MB per step), not flushed: activations and outputs "
              f"stream, the one weight matrix is reused by every row tile anyway")
    return {"workload": w.name, "T": int(w.T), "R": int(w.R),
            "projections": [f"{p.name}:{p.d_in}x{p.d_out}" for p in w.projections],
            "ladder": list(w.policy.ranks), "window": int(w.policy.window), "min_len": int(w.policy.min_len),
            "layers": stack, "n_seq": int(len(w.cu_seqlens) - 1), "steps_include": steps_include, "l2": l2,
            "grouped_launches": bool(grouped), "parallelism": "replicas only" if world > 1 else "single GPU"}


# ----------------------------------------------------------------------------- the oracle, timed
def oracle_sample(w, n_rows: int, n_score_rows: int = 64):
    """Times the fp64 CPU oracle on a bounded sample of the workload; returns (tokens/s, info)."""
    import oracle
    cores = oracle.get_threads()
    p = w.policy
    rng = np.random.default_rng(0)
    t0 = time.perf_counter()
    if w.logits is not None:
        srows = np.sort(rng.choice(w.T, size=min(w.T, n_score_rows), replace=False))
        s_sample = oracle.score_tokens(w.logits[srows])
        t_score = (time.perf_counter() - t0) * (w.T / len(srows))          # scaled to all T rows
        score = np.interp(np.arange(w.T), srows, s_sample).astype(np.float32)  # stand-in track for the partition timing
        ths = np.percentile(s_sample, [25, 50, 75]).astype(np.float32).tolist()
    else:
        srows, t_score, score, ths = [], 0.0, w.score, p.thresholds
    t1 = time.perf_counter()
    if w.table is None:
        tab = oracle.partition(score, w.cu_seqlens, p.ranks, p.scales, ths, p.min_len, p.max_len, p.window, p.hi_budget)
    else:
        t = w.table
        tab = oracle.ChunkTable(t["offsets"], t["rank"], t["scale"], t["rung"], t["flags"], t["n_chunks"])
    t_part = time.perf_counter() - t1
    rows = np.sort(rng.choice(w.T, size=min(n_rows, w.T), replace=False)).astype(np.int32)
    t2 = time.perf_counter()
    for pr in w.projections:
        oracle.apply(w.X[pr.d_in], pr.W, pr.A, pr.B, tab, p.window, rows=rows)
    t_apply_sample = time.perf_counter() - t2
    t_apply = t_apply_sample * (w.T / len(rows))                            # per-row cost is constant
    total = t_score + t_part + t_apply
    info = dict(cores=cores, kind="oracle",
                sample=f"{len(rows)} of {w.T} rows through all {len(w.projections)} projections (fp64 naive loops), "
                       f"score on {len(srows)} rows, partition in full; times scaled to {w.T} rows",
                sample_seconds=time.perf_counter() - t0)
    return w.T / total, info


def rows_for_budget(w, seconds: float):
    """Sample size whose oracle run takes about `seconds` on this host (calibrated on one row per core)."""
    import oracle
    cores = oracle.get_threads()
    t0 = time.perf_counter()
    oracle_sample(w, n_rows=cores, n_score_rows=8)
    t_wave = max(time.perf_counter() - t0, 1e-3)      # one row per core through every projection
    waves = max(1, int(seconds / t_wave))
    return int(min(w.T, cores * waves)), t_wave


def oracle_full_legs(w2=None) -> dict:
    """The oracle timed in full where that takes seconds: the small single-projection configuration end to end,
    on one thread and on all host cores, and the scorer and the chunker on the whole single-sequence prefill
    inputs (2048 x 32000 logits)."""
    import oracle
    from paper_2601_21109_b200 import workloads as wl
    legs = {}
    all_cores = oracle.get_threads()
    w1 = wl.config1()
    p, pr = w1.policy, w1.projections[0]
    for label, n in (("one_thread", 1), ("all_cores", all_cores)):
        oracle.set_threads(n)
        t0 = time.perf_counter()
        tab = oracle.partition(w1.score, w1.cu_seqlens, p.ranks, p.scales, p.thresholds, p.min_len, p.max_len, p.window, p.hi_budget)
        oracle.apply(w1.X[pr.d_in], pr.W, pr.A, pr.B, tab, p.window)
        dt = time.perf_counter() - t0
        legs[f"cfg1_full_{label}"] = {"seconds": dt, "tokens_per_s": w1.T / dt, "threads": n,
                                      "what": "partition + apply, all 256 rows x 1024 columns"}
    if w2 is None:
        w2 = wl.config2()
    p2 = w2.policy
    for label, n in (("one_thread", 1), ("all_cores", all_cores)):
        oracle.set_threads(n)
        t0 = time.perf_counter()
        s = oracle.score_tokens(w2.logits)
        dt = time.perf_counter() - t0
        legs[f"cfg2_score_full_{label}"] = {"seconds": dt, "tokens_per_s": w2.T / dt, "threads": n,
                                            "what": f"cwlo_score_tokens on logits [{w2.T}, {w2.logits.shape[1]}]"}
    oracle.set_threads(all_cores)
    s32 = s.astype(np.float32)
    ths = np.percentile(s32, [25, 50, 75]).astype(np.float32).tolist()
    reps = 20
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle.partition(s32, w2.cu_seqlens, p2.ranks, p2.scales, ths, p2.min_len, p2.max_len, p2.window, p2.hi_budget)
    dt = (time.perf_counter() - t0) / reps
    legs["cfg2_partition_full"] = {"seconds": dt, "tokens_per_s": w2.T / dt, "threads": 1,
                                   "what": f"cwlo_partition on all {w2.T} scores (sequential by definition)"}
    return legs


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = make_workload(args.workload)
    n_layers = layers_of(args.workload, args)
    stack = n_layers if args.workload == "cfg5" else 1
    budget = 150.0 / (args.steps + args.warmup)         # the whole run ends within a few minutes
    n_rows, _ = rows_for_budget(w, budget)
    vals, secs = [], []
    info = {}
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        v, info = oracle_sample(w, n_rows)
        if i >= args.warmup:
            vals.append(v / stack)
            secs.append(time.perf_counter() - t0)
    value = float(np.mean(vals))
    if stack > 1:
        info["sample"] += f"; one layer timed, divided by {stack} layers"
    info["note"] = ("ms_per_step is the wall time of one step's bounded sample; value scales the sample to the whole "
                    "workload (per-row cost is constant)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(args.workload, w, n_layers, args.gpus, not args.no_group),
            "cpu_baseline": dict(value=value, unit=UNIT, **info),
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------- our arm
_T0 = time.time()


def progress(what: str):
    """Phase marks on stderr (stdout carries the one JSON line only)."""
    print(f"[bench +{time.time() - _T0:6.1f}s] {what}", file=sys.stderr, flush=True)


def measure(name: str, args, steps: int, warmup: int, world: int, rank: int, local_rank: int, full: bool):
    """Builds one workload on the device, times it, and returns (result dict, workload)."""
    import torch
    from paper_2601_21109_b200 import binding as cwl
    from paper_2601_21109_b200 import replicas
    from paper_2601_21109_b200 import workloads as wl
    from paper_2601_21109_b200.runner import HotPath

    progress(f"{name}: generating the workload")
    w = make_workload(name)
    n_layers = layers_of(name, args)
    stack = n_layers if name == "cfg5" else 1           # layers one step runs through
    progress(f"{name}: device buffers, plans")
    decode = name in ("cfg4", "cfg4_stream")
    streaming = name == "cfg4_stream"
    hp = HotPath(w, n_layers=n_layers, grouped=not args.no_group, streaming=streaming, prefetch_bytes=int(args.prefetch_mb * 1e6),
                 decode_mode=args.decode_mode)
    stream = torch.cuda.current_stream()

    def barrier():
        replicas.barrier(world)

    def run_step(i: int):
        # a decode step works on ONE weight set, the next step on the next one; a stack step runs every layer
        if decode:
            hp.step(layer=i % n_layers)
        else:
            hp.step()

    # thresholds of the rule-based percentile mapping (Sec. IV-C): quartiles of this batch's scores
    if hp.logits is not None:
        hp.score_step()
        s = hp.score.cpu().numpy()
        hp.set_thresholds(np.percentile(s, [25, 50, 75]).astype(np.float32).tolist())
    run_step(0)
    torch.cuda.synchronize()
    if int(hp.status.item()) != 0:
        raise SystemExit(f"device status word {int(hp.status.item()):#x}")
    table = hp.table.to_host() if not streaming else None
    proj_dims = [(p.d_in, p.d_out) for p in hp.projs]
    if table is not None:
        f_alg, f_exe = table_flops(table, hp.policy.window, hp.T, proj_dims, hp.R)
    else:   # row gates change every step: count the executed (full-rank) work
        f_alg = f_exe = sum(2 * hp.T * di * do + 2 * hp.T * hp.R * (di + do) for di, do in proj_dims)
    f_alg, f_exe = f_alg * stack, f_exe * stack

    # ---- device-resident timing: blocks of `steps` steps, no event inside a block ---------------
    progress(f"{name}: warm-up and timed region")
    for i in range(warmup):
        run_step(i)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(stream)
    for i in range(steps):
        run_step(i)
    b.record(stream)
    torch.cuda.synchronize()
    block_ms = max(a.elapsed_time(b), 1e-3)
    repeats = max(1, int(math.ceil(args.min_seconds * 1e3 / block_ms)))
    if world > 1:
        repeats = int(replicas.max_over_ranks(float(repeats), world))     # every rank runs the same count
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    barrier()
    t_wall0 = time.time()
    marks[0].record(stream)
    for r in range(repeats):
        for i in range(steps):
            run_step(r * steps + i)
        marks[r + 1].record(stream)
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    ms_total = replicas.max_over_ranks(marks[0].elapsed_time(marks[-1]), world)
    block_list = [marks[r].elapsed_time(marks[r + 1]) / steps for r in range(repeats)]
    if int(hp.status.item()) != 0:
        raise SystemExit(f"device status word {int(hp.status.item()):#x}")
    n_steps = steps * repeats
    value = replicas.job_throughput(hp.T, n_steps, world, ms_total)
    ms_per_step = ms_total / n_steps

    progress(f"{name}: apply launches alone, comparison runs")
    # ---- the apply launches alone, inside whole steps (second pass: the headline span above has no inner event) ----
    if decode and not streaming:
        apply_ms = ms_per_step                  # the step IS its apply launches
    else:
        n2 = max(steps, min(n_steps, int(math.ceil(0.5e3 / max(ms_per_step, 1e-3)))))
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n2 * stack)]
        for i in range(n2):
            if streaming:
                hp.stream_state.step(hp.score)
            for layer in range(stack):
                L = (i % n_layers) if decode else layer
                if hp.logits is not None:
                    hp.score_step()
                if not hp.fixed_table and not streaming:
                    hp.partition_step()
                ev[i * stack + layer][0].record(stream)
                hp.apply_step(layer=L)
                ev[i * stack + layer][1].record(stream)
        torch.cuda.synchronize()
        apply_ms = sum(x.elapsed_time(y) for x, y in ev) / n2

    # ---- decode: the same steps under the other schedules (the step's projections side by side on two streams; one after
    # the other on the whole GPU), and, with a fixed table, with the two-stream lanes left running (no join between steps;
    # each lane keeps its order and the region ends with a join: the steps of this workload do not depend on one another,
    # so this is a legal schedule; every other figure keeps step i+1 behind step i).
    free_ms = None
    other_modes = {}
    if decode and not args.lean:
        n3 = max(steps, int(math.ceil(1.0e3 / max(ms_per_step, 1e-3))))
        for mode in ("batch", "lanes", "serial"):
            if mode == hp.decode_mode:
                continue
            alt = HotPath(w, n_layers=n_layers, grouped=not args.no_group, streaming=streaming, share_weights=hp, decode_mode=mode)
            for i in range(10):
                alt.step(layer=i % n_layers)
            x, y = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            x.record(stream)
            for i in range(n3):
                alt.step(layer=i % n_layers)
            y.record(stream)
            torch.cuda.synchronize()
            other_modes[mode] = {"ms_per_step": x.elapsed_time(y) / n3, "steps": n3}
            if mode == "lanes" and not streaming:
                x.record(stream)
                for i in range(n3):
                    alt.apply_step(layer=i % n_layers, join=False, fork=(i == 0))
                alt.join_lanes()
                y.record(stream)
                torch.cuda.synchronize()
                free_ms = x.elapsed_time(y) / n3
            if int(alt.status.item()) != 0:
                raise SystemExit(f"device status word {int(alt.status.item()):#x}")
            del alt

    # ---- comparison runs through the same kernels: static full-rank LoRA and the dense floor ---
    static_ms = dense_ms = chunk_only_ms = None
    if not args.lean:
        st = wl.static_table(w.cu_seqlens, hp.R, 32.0)
        static_tab = cwl.DeviceChunkTable.from_host(st["offsets"], st["rank"], st["scale"], st["flags"], st["rung"])

        def time_apply(**kw):
            est = max(apply_ms, 1e-3)
            n = max(3, int(math.ceil(0.4e3 / est)))
            for i in range(3):
                for layer in range(stack):
                    hp.apply_step(layer=(i % n_layers) if decode else layer, **kw)
            x, y = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            x.record(stream)
            for i in range(n):
                for layer in range(stack):
                    hp.apply_step(layer=(i % n_layers) if decode else layer, **kw)
            y.record(stream)
            torch.cuda.synchronize()
            return x.elapsed_time(y) / n
        chunk_only_ms = time_apply()
        static_ms = time_apply(table=static_tab)
        dense_ms = time_apply(dense=True)

    # ---- end to end: pinned host inputs in, results out, every step ----------------------------
    e2e = None
    if full and not args.lean:
        progress(f"{name}: end to end with host buffers")
        from paper_2601_21109_b200.runner import HostPipeline
        pipe = HostPipeline(w, n_layers=n_layers, grouped=not args.no_group, first=hp, streaming=streaming)
        e2e_steps = max(10, min(steps, 20))    # the span includes one un-overlapped upload and download: ten steps keep them under 5 %
        pipe.run(2)
        barrier()
        x, y = pipe.run(e2e_steps)
        barrier()
        e2e_ms = replicas.max_over_ranks(x.elapsed_time(y), world)
        e2e_value = replicas.job_throughput(hp.T, e2e_steps, world, e2e_ms)
        for slot in pipe.slots:
            if int(slot.status.item()) != 0:
                raise SystemExit(f"device status word {int(slot.status.item()):#x}")
        host_out = pipe.host_Y[0]

        def serial_step():      # the same without overlap (one stream): plain copy - step - copy
            for d, xx in pipe.host_X.items():
                hp.X[d].copy_(xx, non_blocking=True)
            if pipe.host_logits is not None:
                hp.logits.copy_(pipe.host_logits, non_blocking=True)
            if pipe.host_score is not None:
                hp.score.copy_(pipe.host_score, non_blocking=True)
            hp.step()
            for p, yy in zip(hp.projs, host_out):
                yy.copy_(p.Y, non_blocking=True)
        serial_step()
        barrier()
        x, y = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        x.record(stream)
        for _ in range(max(2, e2e_steps // 2)):
            serial_step()
        y.record(stream)
        barrier()
        serial = replicas.job_throughput(hp.T, max(2, e2e_steps // 2), world, replicas.max_over_ranks(x.elapsed_time(y), world))
        e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": pipe.h2d_bytes, "d2h_bytes_per_step": pipe.d2h_bytes,
               "steps": e2e_steps, "serial_value": serial,
               "how": "HostPipeline: two device slots, upload / kernels / download of neighbouring steps overlapped on "
                      "three streams; inputs are copied once per step (a stack step re-scores the same logits in every layer)"}
        del pipe

    # ---- roofline of the dominant kernel (the projection GEMM inside cwl_apply) -----------------
    peaks = load_peaks()
    capped = bool(clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and
                  clocks["sm_mhz"] < 0.9 * clocks["sm_max_mhz"] and "sw_power_cap" in clocks.get("reasons", []))
    if decode:
        bytes_alg = sum(2 * (hp.T * di + di * do + hp.R * (di + do) + hp.T * do) + 2 * hp.T * hp.R * 2 for di, do in proj_dims)
        achieved = bytes_alg / (apply_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": load_traffic("apply_" + name),
                "peak_source": f"hbm copy, of {peaks['source']}", "algorithmic_bytes_per_step": bytes_alg,
                "frac_of_nominal_8000": achieved / 8000.0}
    else:
        # the sustained peak when the sampled clocks show the region ran power-capped, the burst one otherwise
        kind = "bf16_tflops_sustained" if capped else "bf16_tflops"
        achieved = f_alg / (apply_ms * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": peaks[kind], "unit": "TFLOP/s",
                "frac": achieved / peaks[kind], "traffic": load_traffic("apply_" + name),
                "peak_source": f"{kind} ({'power-capped' if capped else 'uncapped'} region by the sampled clocks), of {peaks['source']}",
                "frac_of_burst_peak": achieved / peaks["bf16_tflops"],
                "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"],
                "executed_tflops": f_exe / (apply_ms * 1e-3) / 1e12, "frac_of_nominal_2250": achieved / 2250.0}
    if decode and hp.decode_mode == "batch":
        roof["kernel"] = ("cwl::apply_batch_kernel (the step's projections in one launch, each on its share of the CTA pairs: "
                          "shrink, gate, base GEMM + expand); achieved = the step's algorithmic bytes over the event-timed "
                          "span of its apply launches")
    else:
        roof["kernel"] = ("cwl::apply_kernel (one fused launch per projection or projection group: shrink, gate, base GEMM + "
                          "expand); achieved = the step's algorithmic FLOPs or bytes over the event-timed span of its apply launches")
    roof["launch_ms"] = apply_ms
    roof["sm_mhz_median"] = clocks.get("sm_mhz") if clocks else None
    if clocks and clocks.get("sm_mhz"):
        roof["launch_ms_x_mhz"] = apply_ms * clocks["sm_mhz"]

    res = {"value": value, "unit": UNIT, "ms_per_step": ms_per_step, "ms_per_step_median": float(statistics.median(block_list)),
           "ms_per_step_min": float(min(block_list)), "steps": steps, "inner_repeats": repeats,
           "timed_region_s": ms_total * 1e-3,
           "config": dict(config_dict(name, w, n_layers, world, not args.no_group)),
           "n_chunks": int(table["n_chunks"]) if table is not None else None,
           "tflops": f_alg * n_steps * world / (ms_total * 1e-3) / 1e12,
           "apply_ms_per_step": apply_ms, "apply_only_loop_ms": chunk_only_ms, "decode_mode": hp.decode_mode if decode else None,
           "other_decode_modes": other_modes or None, "free_running_lanes_ms_per_step": free_ms,
           "static_lora_apply_ms": static_ms, "dense_floor_apply_ms": dense_ms,
           "clocks": clocks, "gpu_launches": hp.launches_per_step(stack) * n_steps, "roofline": roof}
    if e2e is not None:
        res["e2e"] = e2e
    del hp
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return res, w


def run_ours(args):
    import torch
    from paper_2601_21109_b200 import binding as cwl
    from paper_2601_21109_b200 import replicas

    rank, local_rank, world = replicas.world_from_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    replicas.init("nccl", local_rank, world)
    cwl.lib()  # fails loudly when libcwl.so is missing

    head, w = measure(args.workload, args, args.steps, args.warmup, world, rank, local_rank, full=True)

    configs, w2 = {}, None
    if world == 1 and not args.lean and not args.no_configs and args.workload == "cfg5":
        for name in SUB_CONFIGS:
            k = {"cfg2": 200, "cfg3": 100, "cfg4": 1000, "cfg4_stream": 1000}[name]
            sub, ws = measure(name, args, k, 5, world, rank, local_rank, full=False)
            if name == "cfg2":
                w2 = ws
            sub["metric"] = METRIC
            configs[name] = sub

    if rank != 0:
        replicas.finish(world)
        return

    stack = head["config"]["layers"]
    if args.lean or world > 1:
        cpu = {}
    else:
        progress("oracle on the host cores")
        n_rows, _ = rows_for_budget(w, 25.0)         # about 10-20 s of CPU work
        cpu_val, cpu_info = oracle_sample(w, n_rows=n_rows)
        if stack > 1:
            cpu_val /= stack
            cpu_info["sample"] += f"; one layer timed, divided by {stack} layers"
        cpu = dict(value=cpu_val, unit=UNIT, **cpu_info)
        cpu["full_runs"] = oracle_full_legs(w2)

    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": head["ms_per_step"], "ms_per_step_median": head["ms_per_step_median"],
        "ms_per_step_min": head["ms_per_step_min"], "inner_repeats": head["inner_repeats"],
        "timed_region_s": head["timed_region_s"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": head["config"], "n_chunks": head["n_chunks"], "tflops": head["tflops"],
        "apply_ms_per_step": head["apply_ms_per_step"], "apply_only_loop_ms": head["apply_only_loop_ms"],
        "static_lora_apply_ms": head["static_lora_apply_ms"], "dense_floor_apply_ms": head["dense_floor_apply_ms"],
        "clocks": head["clocks"], "e2e": head.get("e2e"), "gpu_launches": head["gpu_launches"],
        "roofline": head["roofline"], "cpu_baseline": cpu,
    }
    if configs:
        line["configs"] = configs
    progress("done")
    print(json.dumps(line))
    replicas.finish(world)


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg4_stream", "cfg5"])
    ap.add_argument("--layers", type=int, default=32, help="layers of the cfg5 projection stack (a step runs all of them)")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="least device time of a timed region; the block of --steps steps is repeated until it is reached")
    ap.add_argument("--weight-sets", type=int, default=DECODE_WEIGHT_SETS,
                    help="distinct weight sets a decode run rotates over (4 x 180 MB > L2, so every step streams from HBM)")
    ap.add_argument("--no-configs", action="store_true", help="headline workload only: no `configs` block")
    ap.add_argument("--no-group", action="store_true",
                    help="one cwl_apply launch per projection instead of grouped launches for q,k,v and gate,up")
    ap.add_argument("--decode-mode", default="batch", choices=["batch", "lanes", "serial"],
                    help="decode: the step's projections as one batch launch (default), side by side on two streams, or one "
                         "after the other on one stream, each planned for the whole GPU")
    ap.add_argument("--prefetch-mb", type=float, default=0.0,
                    help="decode: tell each call to pull this many MB of the next call's weights towards L2 while it drains (0: off)")
    ap.add_argument("--lean", action="store_true",
                    help="timed region only (no comparison runs, end-to-end leg or CPU baseline): for profiler runs")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher around us: start one rank per GPU ourselves; rank 0 prints the line
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.run(cmd).returncode)
    if args.impl == "reference":
        args.steps = 2 if args.steps is None else max(1, args.steps)
        args.warmup = 1 if args.warmup is None else max(0, args.warmup)
        run_reference(args)
    else:
        default_steps = {"cfg5": 3, "cfg3": 100, "cfg4": 1000, "cfg4_stream": 1000}.get(args.workload, 200)
        args.steps = default_steps if args.steps is None else max(1, args.steps)
        args.warmup = max(3 if args.warmup is None else args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
