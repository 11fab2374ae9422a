"""Orchestration of one pass of the hot path over a batch: which C calls, in which order.

``HotPath`` keeps the model state resident on the device (weights, adapter factors, workspaces,
the chunk table) and issues score -> partition -> apply for every projection on one stream.  It
contains no arithmetic of the method: thresholds, ladders and windows are handed to the library
as they are.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np
import torch

from . import binding as cwl
from .workloads import Policy, Workload


@dataclass
class DeviceProjection:
    name: str
    d_in: int
    d_out: int
    W: torch.Tensor
    A: torch.Tensor
    B: torch.Tensor
    Y: torch.Tensor


def policy_struct(p: Policy) -> cwl.CPolicy:
    return cwl.make_policy(p.ranks, p.scales, p.thresholds, p.min_len, p.max_len, p.window, p.hi_budget)


class HotPath:
    """Device-resident state of one layer's adapted projections plus the scheduler in front."""

    def __init__(self, w: Workload, device: str = "cuda", keep_host: bool = False, n_layers: int = 1,
                 grouped: bool = True, streaming: bool = False, share_weights: Optional["HotPath"] = None,
                 prefetch_bytes: int = 0, concurrent: bool = True, decode_mode: Optional[str] = None):
        self.grouped = grouped
        self.prefetch_bytes = int(prefetch_bytes)    # decode: bytes of the next call's weights hinted to each call (0 = none)
        # decode with the token-by-token scheduler: every step the cached per-sequence state advances by one
        # token (the rows' scores) and the projections take the row gates it emits instead of a chunk table
        self.streaming = streaming
        self.T, self.R, self.policy = w.T, w.R, w.policy
        self.device = device
        self.cu_seqlens = torch.from_numpy(w.cu_seqlens).to(device)
        self.n_seq = int(w.cu_seqlens.shape[0] - 1)
        self.X: Dict[int, torch.Tensor] = {d: cwl.bf16_from_bits(x, device) for d, x in w.X.items()}
        self.logits = torch.from_numpy(w.logits).to(device) if w.logits is not None else None
        self.score = (torch.from_numpy(w.score).to(device) if w.score is not None
                      else torch.empty(w.T, dtype=torch.float32, device=device))
        self.projs: List[DeviceProjection] = []
        for i, p in enumerate(w.projections):
            if share_weights is not None:      # a second slot of activations and outputs over the same weights
                q = share_weights.projs[i]
                W, A, B = q.W, q.A, q.B
            else:
                W, A, B = cwl.bf16_from_bits(p.W, device), cwl.bf16_from_bits(p.A, device), cwl.bf16_from_bits(p.B, device)
            self.projs.append(DeviceProjection(p.name, p.d_in, p.d_out, W, A, B,
                                               torch.empty(w.T, p.d_out, dtype=torch.bfloat16, device=device)))
        # a stack of layers: every layer has its own weights and adapter factors in HBM (distinct memory, so a
        # layer never finds its weights in L2); layers beyond the first hold the first layer's values rolled by
        # one row per layer, which is all a timing run needs
        self.layers: List[List[DeviceProjection]] = [self.projs]
        for l in range(1, n_layers):
            if share_weights is not None:
                self.layers.append([DeviceProjection(q.name, q.d_in, q.d_out, q.W, q.A, q.B, p.Y)
                                    for q, p in zip(share_weights.layers[l], self.projs)])
                continue
            self.layers.append([DeviceProjection(p.name, p.d_in, p.d_out, torch.roll(p.W, l, 0), torch.roll(p.A, l, 0),
                                                 torch.roll(p.B, l, 1), p.Y) for p in self.projs])
        cap = w.T // max(w.policy.min_len, 1) + self.n_seq + 1
        self.table = cwl.DeviceChunkTable(cap, device)
        if w.table is not None:
            t = w.table
            self.table = cwl.DeviceChunkTable.from_host(t["offsets"], t["rank"], t["scale"], t["flags"], t.get("rung"), device)
        self.fixed_table = w.table is not None
        self.part_ws = torch.empty(cwl.cwl_partition_workspace_bytes(w.T, self.n_seq), dtype=torch.uint8, device=device)
        ws_bytes = max(cwl.cwl_apply_workspace_bytes(w.T, p.d_in, p.d_out, w.R) for p in w.projections)
        for group in self.launch_groups():
            if len(group) > 1:
                ws_bytes = max(ws_bytes, cwl.cwl_apply_grouped_workspace_bytes(
                    w.T, group[0].d_in, [q.d_out for q in group], w.R))
        self.apply_ws = torch.empty(ws_bytes, dtype=torch.uint8, device=device)
        # Decode-sized steps: the projections of a step are independent calls, and each spends a large share of its
        # launch setting up and draining.  They are issued side by side on `lanes` streams, each call planned for its
        # share of the CTA pairs (cwl_set_pair_budget), so that one call's set-up and drain overlap the other's main
        # loop.  Every lane has a workspace of its own.
        # decode_mode: "batch" = the step's projections as ONE launch (cwl_apply_batch: the CTA pairs are shared out among
        # them); "lanes" = side by side on two streams; "serial" = one after the other, each on the whole GPU.
        decode_sized = w.T < self.GROUP_MIN_T and len(w.projections) >= 2
        if decode_mode is None:
            decode_mode = "batch" if concurrent else "serial"
        self.decode_mode = decode_mode if decode_sized else "serial"
        self.batch_calls = None
        if self.decode_mode == "batch":
            n = cwl.MAX_BATCH
            self.batch_calls, self.batch_calls_dense = [], []
            for projs in self.layers:
                groups = [projs[i:i + n] for i in range(0, len(projs), n)]
                self.batch_calls.append([cwl.BatchCall([self.X[p.d_in] for p in g], [p.W for p in g], [p.A for p in g],
                                                       [p.B for p in g], [p.Y for p in g]) for g in groups])
                self.batch_calls_dense.append([cwl.BatchCall([self.X[p.d_in] for p in g], [p.W for p in g], None, None,
                                                             [p.Y for p in g], workspace=c.workspace)
                                               for g, c in zip(groups, self.batch_calls[-1])])
        self.lanes = 2 if self.decode_mode == "lanes" else 1
        if self.lanes > 1:
            self.lane_budget = [self.RESIDENT_PAIRS // self.lanes] * self.lanes
            self.lane_streams = [torch.cuda.Stream(device=device) for _ in range(self.lanes)]
            self.lane_ws = []
            for b in self.lane_budget:
                cwl.cwl_set_pair_budget(b)
                n = max(cwl.cwl_apply_workspace_bytes(w.T, p.d_in, p.d_out, w.R) for p in w.projections)
                self.lane_ws.append(torch.empty(n, dtype=torch.uint8, device=device))
            cwl.cwl_set_pair_budget(0)
            self.fork_event = torch.cuda.Event()
            self.join_events = [torch.cuda.Event() for _ in range(self.lanes)]
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.cpolicy = policy_struct(w.policy)
        self.stream_state = cwl.DeviceStream(w.T, self.cpolicy, device) if streaming else None

    # launches per call, for the benchmark's kernel count
    LAUNCHES_SCORE = 1
    LAUNCHES_PARTITION = 5      # tile sums, prefix, next cut, walk, emit; fewer for small inputs (below)
    LAUNCHES_APPLY = 1          # one fused kernel
    LAUNCHES_APPLY_DENSE = 1

    def set_thresholds(self, thresholds) -> None:
        self.policy.thresholds = [float(np.float32(t)) for t in thresholds]
        self.cpolicy = policy_struct(self.policy)

    def score_step(self) -> None:
        cwl.cwl_score_tokens(self.logits, self.score)

    def partition_step(self) -> None:
        cwl.cwl_partition(self.score, self.cu_seqlens, self.cpolicy, table=self.table, workspace=self.part_ws,
                          status_word=self.status)

    # projections that read the same activation go out as one grouped launch where that is measured to pay: their
    # tiles and shrink items are dealt to the CTA pairs together, which fills the last wave of tiles better than
    # separate calls.  gate + up (2 x 11008 columns) gain from T = 512 on; q + k + v break even at T = 2048 and
    # gain 9 % at T = 8192.  Below GROUP_MIN_T a call is decode-sized: separate calls, whose K loop is split.
    GROUPS = ((("q", "k", "v"), 4096), (("gate", "up"), 512))    # (members, smallest T at which they are grouped)
    GROUP_MIN_T = 512
    RESIDENT_PAIRS = 74          # CTA pairs a B200 holds (148 SMs)

    def launch_groups(self, layer: int = 0) -> List[List[DeviceProjection]]:
        projs = self.layers[layer]
        if not self.grouped or self.T < self.GROUP_MIN_T:
            return [[p] for p in projs]
        by_name = {p.name: p for p in projs}
        out, used = [], set()
        for p in projs:
            if p.name in used:
                continue
            members = next((g for g, min_t in self.GROUPS
                            if p.name in g and self.T >= min_t and all(n in by_name for n in g)), (p.name,))
            out.append([by_name[n] for n in members])
            used.update(members)
        return out

    # Decode-sized calls are bound by HBM and spend a large share of the launch draining (partial sums handed over,
    # outputs stored): each such call is told which weights the NEXT call streams, so that it pulls them towards L2
    # while it drains.  The order of the calls is static (projection after projection, layer after layer).
    PREFETCH_MAX_T = 512

    def _next_weights(self, layer: int, i: int, next_layer: Optional[int]) -> Optional[torch.Tensor]:
        if self.prefetch_bytes <= 0 or self.T >= self.PREFETCH_MAX_T:
            return None
        projs = self.layers[layer]
        if i + 1 < len(projs):
            return projs[i + 1].W
        nl = (layer + 1) % len(self.layers) if next_layer is None else next_layer
        return self.layers[nl][0].W

    def join_lanes(self) -> None:
        """The current stream continues once every lane has finished what it was given."""
        if self.lanes > 1:
            main = torch.cuda.current_stream()
            for ev, st in zip(self.join_events, self.lane_streams):
                ev.record(st)
                main.wait_event(ev)

    def apply_step(self, table: Optional[cwl.DeviceChunkTable] = None, dense: bool = False, layer: int = 0,
                   next_layer: Optional[int] = None, join: bool = True, fork: bool = True) -> None:
        """The adapted projections of one layer.  With lanes, `join=False` leaves the lanes running on their own
        streams (each lane keeps its own order; call join_lanes() before anything reads the outputs) and `fork=False`
        does not make them wait for the current stream again: steps whose projections do not depend on one another
        can then follow one another without draining the GPU in between."""
        rows = self.streaming and table is None and not dense
        tab = table if table is not None else self.table
        if self.batch_calls is not None:
            for call in (self.batch_calls_dense if dense else self.batch_calls)[layer]:
                call(None if (dense or rows) else tab, self.policy.window,
                     gates=self.stream_state.gates if rows else None, status_word=self.status)
            return
        if self.lanes > 1:
            # fork: the lanes start where the current stream stands; join: it continues once every lane is done
            if fork:
                main = torch.cuda.current_stream()
                self.fork_event.record(main)
                for st in self.lane_streams:
                    st.wait_event(self.fork_event)
            try:
                for i, p in enumerate(self.layers[layer]):
                    j = i % self.lanes
                    cwl.cwl_set_pair_budget(self.lane_budget[j])
                    if rows:
                        cwl.cwl_apply_rows(self.X[p.d_in], p.W, p.A, p.B, self.stream_state.gates, Y=p.Y,
                                           workspace=self.lane_ws[j], status_word=self.status, stream=self.lane_streams[j])
                    else:
                        cwl.cwl_apply(self.X[p.d_in], p.W, None if dense else p.A, None if dense else p.B, tab,
                                      self.policy.window, Y=p.Y, workspace=self.lane_ws[j], status_word=self.status,
                                      stream=self.lane_streams[j])
            finally:
                cwl.cwl_set_pair_budget(0)          # later calls of this thread plan for the whole GPU again
            if join:
                self.join_lanes()
            return
        if rows:
            for i, p in enumerate(self.layers[layer]):
                nxt = self._next_weights(layer, i, next_layer)
                if nxt is not None:
                    cwl.cwl_prefetch_next(nxt, self.prefetch_bytes)
                cwl.cwl_apply_rows(self.X[p.d_in], p.W, p.A, p.B, self.stream_state.gates, Y=p.Y,
                                   workspace=self.apply_ws, status_word=self.status)
            return
        for i, group in enumerate(self.launch_groups(layer)):
            p = group[0]
            if len(group) == 1:
                nxt = self._next_weights(layer, i, next_layer)
                if nxt is not None:
                    cwl.cwl_prefetch_next(nxt, self.prefetch_bytes)
                cwl.cwl_apply(self.X[p.d_in], p.W, None if dense else p.A, None if dense else p.B, tab,
                              self.policy.window, Y=p.Y, workspace=self.apply_ws, status_word=self.status)
            else:
                cwl.cwl_apply_grouped(self.X[p.d_in], [q.W for q in group], None if dense else [q.A for q in group],
                                      None if dense else [q.B for q in group], tab, self.policy.window,
                                      Ys=[q.Y for q in group], workspace=self.apply_ws, status_word=self.status)

    def step(self, layer: Optional[int] = None) -> None:
        """One pass of the whole hot path on the current stream (no host synchronisation): through every layer of
        the stack, or, with `layer`, through that weight set alone (decode steps rotate over several sets so that
        no step finds its weights in L2)."""
        if self.streaming:
            self.stream_state.step(self.score)
        for layer in (range(len(self.layers)) if layer is None else (layer,)):
            if self.logits is not None:
                self.score_step()
            if not self.fixed_table:
                self.partition_step()
            self.apply_step(layer=layer)

    def capture(self) -> "torch.cuda.CUDAGraph":
        """Records one step (every launch; a captured apply also records a memset of its sync words) into a CUDA graph.
        The library allocates nothing and synchronises nothing on this path; run one ordinary step first so that
        tensor-map descriptors, plans and kernel attributes are set up outside the capture."""
        self.step()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.step()
        return graph

    def launches_per_step(self, layers: Optional[int] = None) -> int:
        """Kernel launches of one step through `layers` weight sets (default: the whole stack)."""
        n = self.LAUNCHES_APPLY * (len(self.batch_calls[0]) if self.batch_calls is not None else len(self.launch_groups()))
        if self.logits is not None:
            n += self.LAUNCHES_SCORE
        if not self.fixed_table:
            # up to 32 scan tiles of 2048 scores the tile-sum pass is folded into the prefix pass, and a single
            # sequence has its table written by the walk pass
            n += self.LAUNCHES_PARTITION - (1 if self.T <= 32 * 2048 else 0) - (1 if self.n_seq == 1 else 0)
        return n * (len(self.layers) if layers is None else layers) + (1 if self.streaming else 0)


class HostPipeline:
    """End-to-end driver for callers whose inputs and results live in host memory.

    Every step copies that step's inputs (activations, logits) from pinned host buffers to the device, runs
    the hot path and copies all projection outputs back.  Two device slots and three streams (in, compute,
    out) let step i+1's upload and step i-1's download run under step i's kernels, so a step costs the
    slowest of the three instead of their sum.  Weights are shared by the slots."""

    def __init__(self, w: Workload, n_layers: int = 1, grouped: bool = True, device: str = "cuda",
                 first: Optional[HotPath] = None, streaming: bool = False):
        a = first if first is not None else HotPath(w, device, n_layers=n_layers, grouped=grouped, streaming=streaming)
        b = HotPath(w, device, n_layers=n_layers, grouped=grouped, streaming=streaming, share_weights=a)
        b.set_thresholds(a.policy.thresholds) if not a.fixed_table and a.logits is not None else None
        self.slots = [a, b]
        self.host_X = {d: x.cpu().pin_memory() for d, x in a.X.items()}
        self.host_logits = a.logits.cpu().pin_memory() if a.logits is not None else None
        # decode through the scheduler: each slot is its own batch of sequences, and a step's input is one new score
        # per sequence beside the activations
        self.host_score = a.score.cpu().pin_memory() if streaming else None
        self.host_Y = [[torch.empty(p.Y.shape, dtype=p.Y.dtype).pin_memory() for p in s.projs] for s in self.slots]
        self.s_in, self.s_run, self.s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        self.h2d_bytes = sum(x.numel() * x.element_size() for x in self.host_X.values()) + \
            (self.host_logits.numel() * 4 if self.host_logits is not None else 0) + \
            (self.host_score.numel() * 4 if self.host_score is not None else 0)
        self.d2h_bytes = sum(y.numel() * y.element_size() for y in self.host_Y[0])

    def run(self, steps: int):
        """Runs `steps` steps; returns (start, end) CUDA events bracketing the first upload and the last download."""
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        uploaded = [None, None]; computed = [None, None]; downloaded = [None, None]
        self.s_in.wait_stream(torch.cuda.current_stream())
        start.record(self.s_in)
        for i in range(steps):
            k = i & 1
            slot = self.slots[k]
            with torch.cuda.stream(self.s_in):
                if computed[k] is not None:
                    self.s_in.wait_event(computed[k])           # the slot's inputs were consumed
                for d, x in self.host_X.items():
                    slot.X[d].copy_(x, non_blocking=True)
                if self.host_logits is not None:
                    slot.logits.copy_(self.host_logits, non_blocking=True)
                if self.host_score is not None:
                    slot.score.copy_(self.host_score, non_blocking=True)
                uploaded[k] = torch.cuda.Event(); uploaded[k].record(self.s_in)
            with torch.cuda.stream(self.s_run):
                self.s_run.wait_event(uploaded[k])
                if downloaded[k] is not None:
                    self.s_run.wait_event(downloaded[k])        # the slot's outputs were read back
                slot.step()
                computed[k] = torch.cuda.Event(); computed[k].record(self.s_run)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(computed[k])
                for p, y in zip(slot.projs, self.host_Y[k]):
                    y.copy_(p.Y, non_blocking=True)
                downloaded[k] = torch.cuda.Event(); downloaded[k].record(self.s_out)
        self.s_out.wait_stream(self.s_in); self.s_out.wait_stream(self.s_run)
        end.record(self.s_out)
        return start, end
