"""Device timeline of the CTA pairs of a decode step, read with the test build's cwl_trace_set.

    python -m paper_2601_21109_b200.decode_timeline [--mode batch|lanes|serial] [--pairs 0 10 36 37 50 70] [--steps 400]

Builds the decode workload (256 rows, up 4096 x 11008 and down 11008 x 4096, R = 64, four weight sets in rotation),
runs it through the runner exactly as the benchmark does, and for each requested CTA pair traces the leader CTA over
`--steps` steps (the slots keep the last step's readings).  Times are microseconds after the CTA entered the kernel;
%globaltimer ticks every 32 ns.  Tracing adds a global store per K block to the traced pair, so the traced pair runs a
little slower than the others; the step time printed beside it is the event-timed mean of the traced steps.  In a batch
launch pairs are numbered through both projections (0-36 up, 37-73 down); with --mode lanes both launches have a pair of
each number and the slots hold whichever wrote last."""
from __future__ import annotations

import argparse
import ctypes as C

import numpy as np
import torch

from . import binding as cwl
from . import workloads as wl
from .runner import HotPath


def describe(t: np.ndarray) -> list:
    us = lambda i: (int(t[i]) - int(t[0])) / 1e3
    n = int((t[400:690] != 0).sum())
    lines = []
    if n == 0:
        lines.append(f"no work item; launch ahead finished at {us(1):.2f}, teardown {us(4):.2f}")
        return lines
    iss = (t[100:100 + n] - t[0]) / 1e3
    full = (t[400:400 + n] - t[0]) / 1e3
    com = (t[700:700 + n] - t[0]) / 1e3
    period = np.diff(full)[4:] if n > 6 else np.diff(full)
    lines.append(f"K blocks {n}; launch ahead finished {us(1):.2f}; first loads issued {iss[0]:.2f}, landed {full[0]:.2f}; "
                 f"block period mean {period.mean():.3f} median {np.median(period):.3f}; operands landed -> MMAs committed "
                 f"{(com - full)[4:].mean():.3f}; loads issued -> landed mean {(full - iss)[4:].mean():.2f} min {(full - iss).min():.2f}; "
                 f"last block landed {full[-1]:.2f}; accumulator committed {us(2):.2f}; epilogue done {us(3):.2f}; teardown {us(4):.2f}")
    if t[19] != 0:
        lines.append(f"producer: warp past the launch wait {us(19):.2f}, first item decoded {us(20):.2f}, first slot free {us(21):.2f}, first loads issued {iss[0]:.2f}")
    if t[15] != 0:
        lines.append(f"producer waited for H' from {us(15):.2f} to {us(16):.2f}")
    if t[6] != 0:
        lines.append(f"split-K hand-over after the accumulator ({us(5):.2f}): partial sums stored +{(t[6] - t[5]) / 1e3:.2f}, contributors in "
                     f"+{(t[7] - t[6]) / 1e3:.2f}, their sums copied in +{(t[8] - t[7]) / 1e3:.2f}, reduced and staged +{(t[9] - t[8]) / 1e3:.2f}, "
                     f"Y stored +{(t[3] - t[9]) / 1e3:.2f}")
    if t[11] != 0:
        tail = (f", fence passed {us(17):.2f}, partial sums loaded {us(18):.2f}, reduced {us(13):.2f}, fenced {us(14):.2f}"
                if t[13] > t[12] else " (not the last arriver)")
        lines.append(f"shrink epilogue: accumulator seen {us(5):.2f}, partial sums stored and fenced {us(11):.2f}, arrival counted {us(12):.2f}{tail}")
    return lines


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--mode", default="batch", choices=["batch", "lanes", "serial"])
    ap.add_argument("--pairs", type=int, nargs="*", default=[0, 10, 36, 37, 50, 70, 73])
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--weight-sets", type=int, default=4)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    w = wl.config4()
    slots = torch.zeros(1024, dtype=torch.int64, device="cuda")
    with cwl.test_hooks() as L:
        L.cwl_trace_set.restype = C.c_int
        L.cwl_trace_set.argtypes = [C.c_void_p, C.c_int32]
        hp = HotPath(w, n_layers=args.weight_sets, grouped=True, streaming=False, decode_mode=args.mode)
        for i in range(20):
            hp.step(layer=i % args.weight_sets)
        torch.cuda.synchronize()
        for pair in args.pairs:
            slots.zero_()
            torch.cuda.synchronize()
            if L.cwl_trace_set(slots.data_ptr(), pair) != 0:
                raise RuntimeError("cwl_trace_set failed")
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(args.steps):
                hp.step(layer=i % args.weight_sets)
            b.record()
            torch.cuda.synchronize()
            L.cwl_trace_set(None, -1)
            if int(hp.status.item()) != 0:
                raise RuntimeError(f"device status word {int(hp.status.item()):#x}")
            print(f"pair {pair} ({args.mode}; step {a.elapsed_time(b) / args.steps * 1e3:.2f} us):")
            for line in describe(slots.cpu().numpy().astype(np.int64)):
                print("   " + line)


if __name__ == "__main__":
    main()
