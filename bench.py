#!/usr/bin/env python
"""Benchmark of the ChunkWise-LoRA hot path on B200.

One step = one pass of the whole hot path over one batch of the LLaMA-7B-shaped prefill
configuration (T = 2048 tokens): token scoring from fp32 logits [T, 32000], adaptive partition and
rank selection, then the adapted projection for all seven projections (q, k, v, o, gate, up, down)
with R = 64.  Prints ONE JSON line: metric, value (whole-job tokens/s), ms_per_step, config, clocks, e2e (host
buffers in and out every step), gpu_launches, roofline (dominant kernel against the measured peaks) and
cpu_baseline (the fp64 oracle timed on the host cores).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg2|cfg3|cfg4|cfg4_stream|cfg5|cfg1] [--layers L] [--no-group] [--lean]

N > 1 runs N independent replicas (one process per GPU, launched with torch.distributed.run); the
path has no exchange step, so there is no data-path collective: only the timing barrier and the
max-over-ranks reduction of the timed region.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "adapted_projection_tokens_per_s"
UNIT = "tokens/s"


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
APPLY_KERNEL_REVISION = "pairs-256x512-grouped-r6"


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


# ----------------------------------------------------------------------------- reference arm
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


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = make_workload(args.workload)
    budget = 150.0 / (args.steps + args.warmup)         # the whole run ends within a few minutes
    n_rows, _ = rows_for_budget(w, budget)
    vals = []
    info = {}
    for i in range(args.warmup + args.steps):
        v, info = oracle_sample(w, n_rows)
        if i >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * w.T / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "T": w.T, "R": w.R, "projections": [f"{p.name}:{p.d_in}x{p.d_out}" for p in w.projections]},
            "cpu_baseline": dict(value=value, unit=UNIT, **info),
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    from paper_2601_21109_b200 import binding as cwl
    from paper_2601_21109_b200.runner import HotPath

    from paper_2601_21109_b200 import replicas
    rank, local_rank, world = replicas.world_from_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    replicas.init("nccl", local_rank, world)
    cwl.lib()  # fails loudly when libcwl.so is missing

    w = make_workload(args.workload)
    n_layers = args.layers if args.workload == "cfg5" else 1
    streaming = args.workload == "cfg4_stream"
    hp = HotPath(w, n_layers=n_layers, grouped=not args.no_group, streaming=streaming)
    stream = torch.cuda.current_stream()

    # thresholds of the rule-based percentile mapping (Sec. IV-C): quartiles of this batch's scores
    if hp.logits is not None:
        hp.score_step()
        s = hp.score.cpu().numpy()
        hp.set_thresholds(np.percentile(s, [25, 50, 75]).astype(np.float32).tolist())
    hp.step()
    torch.cuda.synchronize()
    if int(hp.status.item()) != 0:
        raise SystemExit(f"device status word {int(hp.status.item()):#x}")
    table = hp.table.to_host()
    proj_dims = [(p.d_in, p.d_out) for p in hp.projs]
    f_alg, f_exe = table_flops(table, hp.policy.window, hp.T, proj_dims, hp.R)
    f_alg, f_exe = f_alg * n_layers, f_exe * n_layers

    def barrier():
        replicas.barrier(world)

    # ---- device-resident timing --------------------------------------------------------------
    for _ in range(args.warmup):
        hp.step()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(args.steps * n_layers)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    barrier()
    t_wall0 = time.time()
    e0.record(stream)
    for i in range(args.steps):
        if streaming:
            hp.stream_state.step(hp.score)
        for layer in range(n_layers):
            if hp.logits is not None:
                hp.score_step()
            if not hp.fixed_table:
                hp.partition_step()
            ev[i * n_layers + layer][0].record(stream)
            hp.apply_step(layer=layer)
            ev[i * n_layers + layer][1].record(stream)
    e1.record(stream)
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    ms_total = e0.elapsed_time(e1)
    apply_ms = [sum(a.elapsed_time(b) for a, b in ev[i * n_layers:(i + 1) * n_layers]) for i in range(args.steps)]
    ms_total = replicas.max_over_ranks(ms_total, world)
    if int(hp.status.item()) != 0:
        raise SystemExit(f"device status word {int(hp.status.item()):#x}")
    value = replicas.job_throughput(hp.T, args.steps, world, ms_total)

    # ---- comparison runs through the same kernels: static full-rank LoRA and the dense floor ---
    from paper_2601_21109_b200 import workloads as wl
    st = wl.static_table(w.cu_seqlens, hp.R, 32.0)
    static_tab = cwl.DeviceChunkTable.from_host(st["offsets"], st["rank"], st["scale"], st["flags"], st["rung"])

    def time_apply(**kw):
        for _ in range(3):
            hp.apply_step(**kw)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = max(3, min(args.steps, 50))
        a.record(stream)
        for _ in range(n):
            for layer in range(n_layers):
                hp.apply_step(layer=layer, **kw)
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n
    static_ms = None if args.lean else time_apply(table=static_tab)
    dense_ms = None if args.lean else time_apply(dense=True)

    # ---- end to end: pinned host inputs in, results out, every step ----------------------------
    # (the library's HostPipeline: uploads, kernels and downloads of neighbouring steps overlap on three streams)
    e2e_value, e2e_serial, e2e_steps, h2d, d2h = None, None, 0, 0, 0
    if not args.lean:
        from paper_2601_21109_b200.runner import HostPipeline
        pipe = HostPipeline(w, n_layers=n_layers, grouped=not args.no_group, first=hp, streaming=streaming)
        h2d, d2h = pipe.h2d_bytes, pipe.d2h_bytes
        e2e_steps = max(4, min(args.steps, 20))
        pipe.run(2)
        barrier()
        a, b = pipe.run(e2e_steps)
        barrier()
        e2e_ms = replicas.max_over_ranks(a.elapsed_time(b), world)
        e2e_value = replicas.job_throughput(hp.T, e2e_steps, world, e2e_ms)
        for slot in pipe.slots:
            if int(slot.status.item()) != 0:
                raise SystemExit(f"device status word {int(slot.status.item()):#x}")
        # the same without overlap (one stream): what a caller gets from plain copy - step - copy
        host_out = pipe.host_Y[0]

        def serial_step():
            for d, x in pipe.host_X.items():
                hp.X[d].copy_(x, non_blocking=True)
            if pipe.host_logits is not None:
                hp.logits.copy_(pipe.host_logits, non_blocking=True)
            if pipe.host_score is not None:
                hp.score.copy_(pipe.host_score, non_blocking=True)
            hp.step()
            for p, y in zip(hp.projs, host_out):
                y.copy_(p.Y, non_blocking=True)
        serial_step()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(e2e_steps):
            serial_step()
        b.record(stream)
        barrier()
        e2e_serial = replicas.job_throughput(hp.T, e2e_steps, world, replicas.max_over_ranks(a.elapsed_time(b), world))

    if rank != 0:
        replicas.finish(world)
        return

    # ---- roofline of the dominant kernel (the projection GEMM inside cwl_apply) -----------------
    peaks = load_peaks()
    apply_avg_ms = float(np.mean(apply_ms))
    region_s = ms_total * 1e-3
    if args.workload in ("cfg4", "cfg4_stream"):
        bytes_alg = sum(2 * (hp.T * di + di * do + hp.R * (di + do) + hp.T * do) + 2 * hp.T * hp.R * 2 for di, do in proj_dims)
        achieved = bytes_alg / (apply_avg_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": load_traffic("apply_" + args.workload),
                "peak_source": f"hbm copy, of {peaks['source']}"}
    else:
        # sustained peak for a long or power-capped region (SM clock pulled well below its maximum), burst otherwise
        capped = bool(clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and
                      clocks["sm_mhz"] < 0.85 * clocks["sm_max_mhz"] and "sw_power_cap" in clocks.get("reasons", []))
        kind = "bf16_tflops_sustained" if (region_s > 1.0 or capped) else "bf16_tflops"
        achieved = f_alg / (apply_avg_ms * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": peaks[kind], "unit": "TFLOP/s",
                "frac": achieved / peaks[kind], "traffic": load_traffic("apply_" + args.workload),
                "peak_source": f"{kind}, of {peaks['source']}"}
    roof["kernel"] = ("cwl::apply_kernel (one fused launch per projection: shrink, gate, base GEMM + expand); achieved = the "
                      "step's algorithmic FLOPs or bytes over the event-timed span of its apply launches")
    if roof["bound"] == "tensor":
        roof["frac_of_burst_peak"] = roof["achieved"] / peaks["bf16_tflops"]
        roof["frac_of_sustained_peak"] = roof["achieved"] / peaks["bf16_tflops_sustained"]
    roof["launch_ms"] = apply_avg_ms
    roof["executed_tflops"] = f_exe / (apply_avg_ms * 1e-3) / 1e12
    roof["frac_of_nominal_2250"] = (f_alg / (apply_avg_ms * 1e-3) / 1e12) / 2250.0

    parts = (["scheduler step"] if streaming else []) + (["score"] if hp.logits is not None else []) + ([] if hp.fixed_table else ["partition"]) + \
        [f"{len(hp.projs)} projections in {len(hp.launch_groups())} apply launches"]
    steps_include = (f"{n_layers} layers x (" if n_layers > 1 else "(") + " + ".join(parts) + ")"
    step_bytes = n_layers * (sum(2 * p.d_in * p.d_out for p in hp.projs) +
                             (hp.logits.numel() * 4 if hp.logits is not None else 0))
    l2_note = (f"inputs larger than L2 ({step_bytes / 1e6:.0f} MB of weights and logits read per step)"
               if step_bytes > 126e6 else
               f"inputs smaller than L2 ({step_bytes / 1e6:.1f} MB per step), not flushed: parity-sized workload, not a headline")
    if args.lean:
        cpu_val, cpu_info = None, {}
    else:
        n_rows, _ = rows_for_budget(w, 12.0)         # about 10-20 s of CPU work
        cpu_val, cpu_info = oracle_sample(w, n_rows=n_rows)
        if n_layers > 1:
            cpu_val /= n_layers
            cpu_info["sample"] += f"; one layer timed, divided by {n_layers} layers"

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "T": hp.T, "R": hp.R, "projections": [f"{p.name}:{p.d_in}x{p.d_out}" for p in hp.projs],
                   "ladder": hp.policy.ranks, "window": hp.policy.window, "min_len": hp.policy.min_len,
                   "n_chunks": table["n_chunks"], "layers": n_layers, "steps_include": steps_include, "l2": l2_note,
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "tflops": f_alg * args.steps * world / (ms_total * 1e-3) / 1e12,
        "apply_ms_per_step": apply_avg_ms,
        "static_lora_apply_ms": static_ms, "dense_floor_apply_ms": dense_ms,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "how": "HostPipeline: two device slots, upload / kernels / download of neighbouring steps overlapped on three streams",
                "serial_value": e2e_serial},
        "gpu_launches": hp.launches_per_step() * args.steps,
        "roofline": roof,
        "cpu_baseline": dict(value=cpu_val, unit=UNIT, **cpu_info),
    }
    print(json.dumps(line))
    replicas.finish(world)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg4_stream", "cfg5"])
    ap.add_argument("--layers", type=int, default=32, help="layers of the cfg5 projection stack (a step runs all of them)")
    ap.add_argument("--no-group", action="store_true",
                    help="one cwl_apply launch per projection instead of grouped launches for q,k,v and gate,up")
    ap.add_argument("--lean", action="store_true",
                    help="timed region only (no comparison runs, end-to-end leg or CPU baseline): for profiler runs")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 2 if args.steps is None else max(1, args.steps)
        args.warmup = 1 if args.warmup is None else max(0, args.warmup)
        run_reference(args)
    else:
        default_steps = {"cfg5": 5, "cfg3": 100}.get(args.workload, 500)
        args.steps = default_steps if args.steps is None else max(1, args.steps)
        args.warmup = max(5 if args.warmup is None else args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
