"""Read-bandwidth ceiling of a decode-sized launch, measured with the test build's cwl_probe_read.

    python -m paper_2601_21109_b200.read_ceiling [--mb 33.5 90.2 180.4 360.7] [--seconds 1.0]
    python -m paper_2601_21109_b200.read_ceiling --mb 180.4 --mix 0 5376 10752 16384 --ctas 148 124   (cwl_probe_read_mix)

For every size: back-to-back launches (chained like the apply kernel's) rotate over enough distinct regions to
exceed L2 several times, so every launch reads from HBM; CUDA events bracket the whole loop.  One launch = 148
CTAs, each streaming its slice through a 192 KB shared-memory ring with 16 KB bulk copies and dropping the data.
Prints microseconds per launch and GB/s; the figure for 90 MB (the bytes of one 4096 x 11008 bf16 projection) is
what a decode launch could reach if its tensor-core work, hand-over and output stores cost nothing."""
from __future__ import annotations

import argparse
import ctypes as C
import json
import math

import torch

from . import binding as cwl


def measure(mb: float, seconds: float) -> dict:
    n_bytes = int(mb * 1e6) // (148 * 16384) * (148 * 16384)
    n_regions = max(4, int(math.ceil(600e6 / n_bytes)))            # >= 600 MB in rotation: several times L2
    regions = [torch.empty(n_bytes, dtype=torch.uint8, device="cuda").fill_(i + 1) for i in range(n_regions)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    with cwl.test_hooks() as L:
        L.cwl_probe_read.restype = C.c_int
        L.cwl_probe_read.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]

        def launch(i):
            rc = L.cwl_probe_read(regions[i % n_regions].data_ptr(), n_bytes, status.data_ptr(), stream.cuda_stream)
            if rc != 0:
                raise RuntimeError(f"cwl_probe_read: status {rc}")
        for i in range(2 * n_regions):
            launch(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(20):
            launch(i)
        b.record()
        torch.cuda.synchronize()
        n = max(20, int(seconds * 1e3 / max(a.elapsed_time(b) / 20, 1e-3)))
        a.record()
        for i in range(n):
            launch(i)
        b.record()
        torch.cuda.synchronize()
    if int(status.item()) != 0:
        raise RuntimeError(f"device status word {int(status.item()):#x}")
    us = a.elapsed_time(b) * 1e3 / n
    return {"mb": n_bytes / 1e6, "regions": n_regions, "launches": n, "us_per_launch": us, "gb_per_s": n_bytes / us / 1e3}


def measure_mix(mb: float, seconds: float, hot_piece: int, ctas: int, hot_mb: float = 2.0) -> dict:
    """The stream of `measure` with `hot_piece` bytes out of a small L2-resident region copied beside every 16 KB piece,
    on `ctas` CTAs: the mix of HBM and L2 traffic the apply kernel's K loop has (24 KB of W and 16 KB of X per stage
    = 10.7 KB of X per 16 KB of W)."""
    n_bytes = int(mb * 1e6) // (ctas * 16384) * (ctas * 16384)
    n_regions = max(4, int(math.ceil(600e6 / n_bytes)))
    regions = [torch.empty(n_bytes, dtype=torch.uint8, device="cuda").fill_(i + 1) for i in range(n_regions)]
    hot = torch.empty(int(hot_mb * 1e6) // hot_piece * hot_piece, dtype=torch.uint8, device="cuda").fill_(7)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    with cwl.test_hooks() as L:
        L.cwl_probe_read_mix.restype = C.c_int
        L.cwl_probe_read_mix.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_uint32, C.c_int32, C.c_void_p, C.c_void_p]

        def launch(i):
            rc = L.cwl_probe_read_mix(regions[i % n_regions].data_ptr(), n_bytes, hot.data_ptr(), hot.numel(), hot_piece, ctas,
                                      status.data_ptr(), stream.cuda_stream)
            if rc != 0:
                raise RuntimeError(f"cwl_probe_read_mix: status {rc}")
        for i in range(2 * n_regions):
            launch(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(20):
            launch(i)
        b.record()
        torch.cuda.synchronize()
        n = max(20, int(seconds * 1e3 / max(a.elapsed_time(b) / 20, 1e-3)))
        a.record()
        for i in range(n):
            launch(i)
        b.record()
        torch.cuda.synchronize()
    if int(status.item()) != 0:
        raise RuntimeError(f"device status word {int(status.item()):#x}")
    us = a.elapsed_time(b) * 1e3 / n
    hot_total = n_bytes // 16384 * hot_piece
    return {"mb": n_bytes / 1e6, "ctas": ctas, "hot_piece": hot_piece, "hot_mb_per_launch": hot_total / 1e6, "launches": n,
            "us_per_launch": us, "hbm_gb_per_s": n_bytes / us / 1e3, "delivered_gb_per_s": (n_bytes + hot_total) / us / 1e3}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--mb", type=float, nargs="*", default=[33.6, 90.2, 180.4, 360.7])
    ap.add_argument("--seconds", type=float, default=1.0)
    ap.add_argument("--mix", type=int, nargs="*", default=None,
                    help="bytes of an L2-resident region copied beside every 16 KB piece (multiples of 16), e.g. 0 5376 10752 16384")
    ap.add_argument("--ctas", type=int, nargs="*", default=[148], help="CTAs of the mixed read (1..148)")
    args = ap.parse_args()
    if args.mix is not None:
        for mb in args.mb:
            for ctas in args.ctas:
                for hot_piece in args.mix:
                    if hot_piece == 0 and ctas == 148:
                        print(json.dumps(measure(mb, args.seconds)))
                    elif hot_piece > 0:
                        print(json.dumps(measure_mix(mb, args.seconds, hot_piece, ctas)))
        return
    for mb in args.mb:
        print(json.dumps(measure(mb, args.seconds)))


if __name__ == "__main__":
    main()
