"""ctypes binding of libcwl.so: argument marshalling only.

Every step of the path (scoring, partition, shrink, gate, projection) runs in the CUDA library;
torch is used for device memory and streams.  There is no CPU fallback: if the library has not
been built, loading raises.  Function names mirror the C ABI declared in ``include/cwl.h``.
"""
from __future__ import annotations

import contextlib
import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcwl.so")
MAX_RUNGS = 8

STATUS = {0: "CWL_OK", 1: "CWL_ERR_INVALID_ARG", 2: "CWL_ERR_SHAPE", 3: "CWL_ERR_UNSUPPORTED",
          4: "CWL_ERR_CAPACITY", 5: "CWL_ERR_WORKSPACE", 6: "CWL_ERR_CUDA", 7: "CWL_ERR_TIMEOUT"}

EXPORTS = ["cwl_status_string", "cwl_version", "cwl_score_tokens", "cwl_score_tokens_mixed", "cwl_partition_workspace_bytes",
           "cwl_partition", "cwl_apply_workspace_bytes", "cwl_apply", "cwl_apply_grouped_workspace_bytes",
           "cwl_apply_grouped", "cwl_apply_plan", "cwl_stream_state_bytes", "cwl_stream_reset", "cwl_stream_step",
           "cwl_apply_rows", "cwl_ladder_workspace_bytes", "cwl_ladder_build",
           "cwl_apply_noalloc_scratch_need", "cwl_apply_noalloc", "cwl_prefetch_next", "cwl_apply_mode",
           "cwl_batch_align_workspace_bytes", "cwl_batch_align", "cwl_set_pair_budget",
           "cwl_apply_batch_workspace_bytes", "cwl_apply_batch"]
NOALLOC_SCRATCH_BYTES = 8 << 20
WINDOW_CAUSAL, WINDOW_CENTRED = 0, 1
MAX_BATCH = 4


class CwlError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        super().__init__(f"{call} failed: {STATUS.get(status, status)}")


class CPolicy(C.Structure):
    _fields_ = [("n_rungs", C.c_int32),
                ("rung_rank", C.c_int32 * MAX_RUNGS),
                ("rung_scale", C.c_float * MAX_RUNGS),
                ("threshold", C.c_float * (MAX_RUNGS - 1)),
                ("min_len", C.c_int32), ("max_len", C.c_int32),
                ("window", C.c_int32), ("hi_budget", C.c_int32)]


class CChunkTable(C.Structure):
    _fields_ = [("offsets", C.c_void_p), ("rank", C.c_void_p), ("scale", C.c_void_p),
                ("rung", C.c_void_p), ("flags", C.c_void_p), ("n_chunks", C.c_void_p),
                ("capacity", C.c_int32)]


MAX_GROUP = 4
STREAM_MAX_MIN_LEN = 64


class CRowGate(C.Structure):
    _fields_ = [("rank_in", C.c_int32), ("rank_out", C.c_int32), ("scale_in", C.c_float), ("scale_out", C.c_float),
                ("lam", C.c_float), ("pos_in_chunk", C.c_int32), ("opened", C.c_int32)]


ROW_GATE_BYTES = C.sizeof(CRowGate)     # 28: gates live in a uint8 tensor of [n, ROW_GATE_BYTES]


class CProjection(C.Structure):
    _fields_ = [("W", C.c_void_p), ("ldw", C.c_int64), ("A", C.c_void_p), ("lda", C.c_int64),
                ("B", C.c_void_p), ("ldb", C.c_int64), ("Y", C.c_void_p), ("ldy", C.c_int64), ("d_out", C.c_int32)]


class CBatchItem(C.Structure):
    _fields_ = [("X", C.c_void_p), ("ldx", C.c_int64), ("d_in", C.c_int32),
                ("W", C.c_void_p), ("ldw", C.c_int64), ("A", C.c_void_p), ("lda", C.c_int64),
                ("B", C.c_void_p), ("ldb", C.c_int64), ("Y", C.c_void_p), ("ldy", C.c_int64), ("d_out", C.c_int32)]


class CSignalMix(C.Structure):
    _fields_ = [("w_entropy", C.c_float), ("w_novelty", C.c_float), ("w_prior", C.c_float),
                ("ngram", C.c_int32), ("context", C.c_int32), ("prior_span", C.c_int32)]


class CApplyPlanInfo(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "pairs", "row_tiles", "wide_width", "wide_tiles_per_row", "narrow_width", "narrow_tiles_per_row",
        "split_k", "k_blocks_per_split", "shrink_splits", "shrink_items", "shrink_items_assigned",
        "shrink_items_max_per_pair", "stages")] + [("model_cost", C.c_int64)]


_lib = None
_hooks_lib = None
HOOKS_LIB_PATH = os.path.join(_HERE, "libcwl_hooks.so")


def lib():
    """Loads libcwl.so (built by ``paper_2601_21109_b200.build``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2601_21109_b200.build` "
                               "(there is no fallback path)")
        _lib = _declare(C.CDLL(LIB_PATH))
    return _lib


@contextlib.contextmanager
def test_hooks():
    """Routes every call of this module through the TEST build of the library (libcwl_hooks.so: the same sources
    compiled with -DCWL_TEST_HOOKS, which adds cwl_debug_set) for the duration of the block."""
    global _lib, _hooks_lib
    if _hooks_lib is None:
        if not os.path.exists(HOOKS_LIB_PATH):
            raise RuntimeError(f"{HOOKS_LIB_PATH} is missing: run `python -m paper_2601_21109_b200.build`")
        _hooks_lib = _declare(C.CDLL(HOOKS_LIB_PATH))
        _hooks_lib.cwl_debug_set.restype = None
        _hooks_lib.cwl_debug_set.argtypes = [C.c_int64, C.c_int32]
    saved = lib()
    _lib = _hooks_lib
    try:
        yield _hooks_lib
    finally:
        _hooks_lib.cwl_debug_set(0, 0)
        _lib = saved


def _declare(L):
    """Argument and result types of every exported call."""
    if True:
        L.cwl_status_string.restype = C.c_char_p
        L.cwl_status_string.argtypes = [C.c_int]
        L.cwl_version.restype = C.c_int
        L.cwl_score_tokens.restype = C.c_int
        L.cwl_score_tokens.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.cwl_score_tokens_mixed.restype = C.c_int
        L.cwl_score_tokens_mixed.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                             C.c_int32, C.POINTER(CSignalMix), C.c_void_p, C.c_void_p]
        L.cwl_partition_workspace_bytes.restype = C.c_size_t
        L.cwl_partition_workspace_bytes.argtypes = [C.c_int32, C.c_int32]
        L.cwl_partition.restype = C.c_int
        L.cwl_partition.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.POINTER(CPolicy), CChunkTable,
                                    C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.cwl_batch_align_workspace_bytes.restype = C.c_size_t
        L.cwl_batch_align_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        L.cwl_batch_align.restype = C.c_int
        L.cwl_batch_align.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.POINTER(CPolicy), C.c_int32,
                                      CChunkTable, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.cwl_apply_workspace_bytes.restype = C.c_size_t
        L.cwl_apply_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32]
        L.cwl_apply.restype = C.c_int
        L.cwl_apply.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                CChunkTable, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t,
                                C.c_void_p, C.c_void_p]
        L.cwl_apply_mode.restype = C.c_int
        L.cwl_apply_mode.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                     C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32, CChunkTable,
                                     C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.cwl_apply_grouped_workspace_bytes.restype = C.c_size_t
        L.cwl_apply_grouped_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_int32), C.c_int32]
        L.cwl_apply_grouped.restype = C.c_int
        L.cwl_apply_grouped.argtypes = [C.c_void_p, C.c_int64, C.POINTER(CProjection), C.c_int32, C.c_int32, C.c_int32,
                                        C.c_int32, CChunkTable, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.cwl_stream_state_bytes.restype = C.c_size_t
        L.cwl_stream_state_bytes.argtypes = [C.c_int32, C.c_int32]
        L.cwl_stream_reset.restype = C.c_int
        L.cwl_stream_reset.argtypes = [C.c_void_p, C.c_size_t, C.c_int32, C.c_int32, C.c_void_p]
        L.cwl_stream_step.restype = C.c_int
        L.cwl_stream_step.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(CPolicy), C.c_void_p, C.c_size_t,
                                      C.c_void_p, C.c_void_p]
        L.cwl_apply_rows.restype = C.c_int
        L.cwl_apply_rows.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                     C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                     C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.cwl_ladder_workspace_bytes.restype = C.c_size_t
        L.cwl_ladder_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        L.cwl_ladder_build.restype = C.c_int
        L.cwl_ladder_build.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                       C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_size_t, C.POINTER(C.c_int32), C.c_void_p]
        L.cwl_apply_batch_workspace_bytes.restype = C.c_size_t
        L.cwl_apply_batch_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_int32]
        L.cwl_apply_batch.restype = C.c_int
        L.cwl_apply_batch.argtypes = [C.POINTER(CBatchItem), C.c_int32, C.c_int32, C.c_int32, CChunkTable, C.c_void_p, C.c_int32,
                                      C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.cwl_set_pair_budget.restype = C.c_int
        L.cwl_set_pair_budget.argtypes = [C.c_int32]
        L.cwl_prefetch_next.restype = C.c_int
        L.cwl_prefetch_next.argtypes = [C.c_void_p, C.c_size_t]
        L.cwl_apply_plan.restype = C.c_int
        L.cwl_apply_plan.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(CApplyPlanInfo)]
        L.cwl_apply_noalloc_scratch_need.restype = C.c_size_t
        L.cwl_apply_noalloc_scratch_need.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32]
        L.cwl_apply_noalloc.restype = C.c_int
        L.cwl_apply_noalloc.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                        C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                        CChunkTable, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
    return L


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _p(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def make_policy(ranks: Sequence[int], scales: Sequence[float], thresholds: Sequence[float],
                min_len: int, max_len: int, window: int, hi_budget: int = -1) -> CPolicy:
    p = CPolicy()
    p.n_rungs = len(ranks)
    for k, r in enumerate(ranks):
        p.rung_rank[k] = int(r)
    for k, s in enumerate(scales):
        p.rung_scale[k] = float(s)
    for k, th in enumerate(thresholds):
        p.threshold[k] = float(th)
    p.min_len, p.max_len, p.window, p.hi_budget = int(min_len), int(max_len), int(window), int(hi_budget)
    return p


class DeviceChunkTable:
    """Chunk table as device arrays (struct of arrays, as the C ABI takes it)."""

    def __init__(self, capacity: int, device="cuda"):
        self.capacity = int(capacity)
        self.offsets = torch.zeros(self.capacity + 1, dtype=torch.int32, device=device)
        self.rank = torch.zeros(max(self.capacity, 1), dtype=torch.int32, device=device)
        self.scale = torch.zeros(max(self.capacity, 1), dtype=torch.float32, device=device)
        self.rung = torch.zeros(max(self.capacity, 1), dtype=torch.int32, device=device)
        self.flags = torch.zeros(max(self.capacity, 1), dtype=torch.int32, device=device)
        self.n_chunks = torch.zeros(1, dtype=torch.int32, device=device)

    @staticmethod
    def from_host(offsets, rank, scale, flags, rung=None, device="cuda") -> "DeviceChunkTable":
        n = len(rank)
        t = DeviceChunkTable(n, device)
        t.offsets.copy_(torch.as_tensor(offsets, dtype=torch.int32))
        if n:
            t.rank[:n].copy_(torch.as_tensor(rank, dtype=torch.int32))
            t.scale[:n].copy_(torch.as_tensor(scale, dtype=torch.float32))
            t.flags[:n].copy_(torch.as_tensor(flags, dtype=torch.int32))
            if rung is not None:
                t.rung[:n].copy_(torch.as_tensor(rung, dtype=torch.int32))
        t.n_chunks.fill_(n)
        return t

    def c_struct(self) -> CChunkTable:
        return CChunkTable(_p(self.offsets), _p(self.rank), _p(self.scale), _p(self.rung), _p(self.flags),
                           _p(self.n_chunks), self.capacity)

    def to_host(self) -> dict:
        n = int(self.n_chunks.item())
        return dict(offsets=self.offsets[:n + 1].cpu().numpy(), rank=self.rank[:n].cpu().numpy(),
                    scale=self.scale[:n].cpu().numpy(), rung=self.rung[:n].cpu().numpy(),
                    flags=self.flags[:n].cpu().numpy(), n_chunks=n)


def _check(call: str, status: int) -> None:
    if status != 0:
        raise CwlError(call, status)


def cwl_score_tokens(logits: torch.Tensor, score: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """score[t] = normalised softmax entropy of logits[t, :] (fp32 [T, V] on the device)."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.dim() == 2 and logits.stride(1) == 1
    T, V = logits.shape
    if score is None:
        score = torch.empty(T, dtype=torch.float32, device=logits.device)
    _check("cwl_score_tokens", lib().cwl_score_tokens(_p(logits), logits.stride(0) if T > 1 else max(V, logits.stride(0)),
                                                      T, V, _p(score), _stream_ptr(stream)))
    return score


def cwl_score_tokens_mixed(logits: torch.Tensor, token_ids: torch.Tensor, cu_seqlens: torch.Tensor,
                           w_entropy: float, w_novelty: float, w_prior: float, ngram: int, context: int,
                           prior_span: int, score: Optional[torch.Tensor] = None,
                           stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Entropy, n-gram novelty and positional prior mixed into one score per token (one kernel)."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.dim() == 2 and logits.stride(1) == 1
    assert token_ids.is_cuda and token_ids.dtype == torch.int32 and token_ids.is_contiguous()
    assert cu_seqlens.is_cuda and cu_seqlens.dtype == torch.int32 and cu_seqlens.is_contiguous()
    T, V = logits.shape
    if score is None:
        score = torch.empty(T, dtype=torch.float32, device=logits.device)
    mix = CSignalMix(float(w_entropy), float(w_novelty), float(w_prior), int(ngram), int(context), int(prior_span))
    _check("cwl_score_tokens_mixed", lib().cwl_score_tokens_mixed(
        _p(logits), logits.stride(0) if T > 1 else max(V, logits.stride(0)), T, V, _p(token_ids), _p(cu_seqlens),
        cu_seqlens.numel() - 1, C.byref(mix), _p(score), _stream_ptr(stream)))
    return score


def cwl_partition_workspace_bytes(T: int, n_seq: int) -> int:
    return int(lib().cwl_partition_workspace_bytes(T, n_seq))


def cwl_partition(score: torch.Tensor, cu_seqlens: torch.Tensor, policy: CPolicy,
                  table: Optional[DeviceChunkTable] = None, workspace: Optional[torch.Tensor] = None,
                  status_word: Optional[torch.Tensor] = None,
                  stream: Optional[torch.cuda.Stream] = None) -> DeviceChunkTable:
    """Adaptive chunker + rank-ladder selector; the table stays on the device."""
    assert score.is_cuda and score.dtype == torch.float32 and score.is_contiguous()
    assert cu_seqlens.is_cuda and cu_seqlens.dtype == torch.int32 and cu_seqlens.is_contiguous()
    T, n_seq = score.shape[0], cu_seqlens.shape[0] - 1
    if table is None:
        table = DeviceChunkTable(T // max(int(policy.min_len), 1) + n_seq + 1, score.device)
    need = cwl_partition_workspace_bytes(T, n_seq)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=score.device)
    _check("cwl_partition", lib().cwl_partition(_p(score), _p(cu_seqlens), n_seq, T, C.byref(policy),
                                                table.c_struct(), _p(workspace), workspace.numel(),
                                                _p(status_word), _stream_ptr(stream)))
    return table


def cwl_batch_align(score: torch.Tensor, cu_seqlens: torch.Tensor, policy: CPolicy, n_buckets: int,
                    table: Optional[DeviceChunkTable] = None, workspace: Optional[torch.Tensor] = None,
                    status_word: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Batch alignment: sequences bucketed by complexity percentile share their chunk joins.
    Returns (table, bucket [n_seq] int32, order_pos [n_seq] int32), all on the device."""
    assert score.is_cuda and score.dtype == torch.float32 and score.is_contiguous()
    assert cu_seqlens.is_cuda and cu_seqlens.dtype == torch.int32 and cu_seqlens.is_contiguous()
    T, n_seq = score.shape[0], cu_seqlens.shape[0] - 1
    if table is None:
        table = DeviceChunkTable(T // max(int(policy.min_len), 1) + n_seq + 1, score.device)
    bucket = torch.empty(max(n_seq, 1), dtype=torch.int32, device=score.device)
    order_pos = torch.empty(max(n_seq, 1), dtype=torch.int32, device=score.device)
    if workspace is None:
        workspace = torch.empty(max(16, int(lib().cwl_batch_align_workspace_bytes(T, n_seq, n_buckets))), dtype=torch.uint8,
                                device=score.device)
    _check("cwl_batch_align", lib().cwl_batch_align(_p(score), _p(cu_seqlens), n_seq, T, C.byref(policy), int(n_buckets),
                                                    table.c_struct(), _p(bucket), _p(order_pos), _p(workspace),
                                                    workspace.numel(), _p(status_word), _stream_ptr(stream)))
    return table, bucket[:n_seq], order_pos[:n_seq]


def cwl_apply_workspace_bytes(T: int, d_in: int, d_out: int, R: int) -> int:
    return int(lib().cwl_apply_workspace_bytes(T, d_in, d_out, R))


def cwl_apply_plan(T: int, d_in: int, d_out: int, R: int, pairs: int = 74) -> dict:
    """The schedule cwl_apply would use for this shape with `pairs` resident CTA pairs (host only)."""
    info = CApplyPlanInfo()
    _check("cwl_apply_plan", lib().cwl_apply_plan(T, d_in, d_out, R, pairs, C.byref(info)))
    return {name: int(getattr(info, name)) for name, _ in CApplyPlanInfo._fields_}


def cwl_apply_noalloc_scratch_need(T: int, d_in: int, d_out: int, R: int) -> int:
    return int(lib().cwl_apply_noalloc_scratch_need(T, d_in, d_out, R))


def cwl_apply(X: torch.Tensor, W: torch.Tensor, A: Optional[torch.Tensor], B: Optional[torch.Tensor],
              table: Optional[DeviceChunkTable], window: int, Y: Optional[torch.Tensor] = None,
              workspace: Optional[torch.Tensor] = None, status_word: Optional[torch.Tensor] = None,
              stream: Optional[torch.cuda.Stream] = None, centred: bool = False) -> torch.Tensor:
    """Y = X W + gated (X A) B per the chunk table (bf16 tensors on the device, row-major).  ``centred`` places the
    cross-fade window around each join (cwl_apply_mode) instead of after it."""
    for t in (X, W):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.dim() == 2 and t.stride(1) == 1
    T, d_in = X.shape
    d_out = W.shape[1]
    R = 0
    if A is not None and B is not None:
        assert A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16 and A.stride(1) == 1 and B.stride(1) == 1
        R = A.shape[1]
    if Y is None:
        Y = torch.empty(T, d_out, dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = torch.empty(cwl_apply_workspace_bytes(T, d_in, d_out, R), dtype=torch.uint8, device=X.device)
    ct = table.c_struct() if table is not None else CChunkTable(None, None, None, None, None, None, 0)
    if centred:
        _check("cwl_apply_mode", lib().cwl_apply_mode(_p(X), X.stride(0), _p(W), W.stride(0),
                                                      _p(A), A.stride(0) if R else 0, _p(B), B.stride(0) if R else 0,
                                                      T, d_in, d_out, R, ct, int(window), WINDOW_CENTRED, _p(Y), Y.stride(0),
                                                      _p(workspace), workspace.numel(), _p(status_word), _stream_ptr(stream)))
        return Y
    _check("cwl_apply", lib().cwl_apply(_p(X), X.stride(0), _p(W), W.stride(0),
                                        _p(A), A.stride(0) if R else 0, _p(B), B.stride(0) if R else 0,
                                        T, d_in, d_out, R, ct, int(window), _p(Y), Y.stride(0),
                                        _p(workspace), workspace.numel(), _p(status_word), _stream_ptr(stream)))
    return Y


def cwl_apply_grouped_workspace_bytes(T: int, d_in: int, d_outs: Sequence[int], R: int) -> int:
    arr = (C.c_int32 * len(d_outs))(*[int(d) for d in d_outs])
    return int(lib().cwl_apply_grouped_workspace_bytes(T, d_in, len(d_outs), arr, R))


def cwl_apply_grouped(X: torch.Tensor, Ws: Sequence[torch.Tensor], As: Optional[Sequence[torch.Tensor]],
                      Bs: Optional[Sequence[torch.Tensor]], table: Optional[DeviceChunkTable], window: int,
                      Ys: Optional[Sequence[torch.Tensor]] = None, workspace: Optional[torch.Tensor] = None,
                      status_word: Optional[torch.Tensor] = None,
                      stream: Optional[torch.cuda.Stream] = None) -> Sequence[torch.Tensor]:
    """Y_j = X W_j + gated (X A_j) B_j for up to four projections of the same rows, one launch."""
    T, d_in = X.shape
    n = len(Ws)
    R = As[0].shape[1] if (As is not None and Bs is not None) else 0
    if Ys is None:
        Ys = [torch.empty(T, W.shape[1], dtype=torch.bfloat16, device=X.device) for W in Ws]
    if workspace is None:
        workspace = torch.empty(cwl_apply_grouped_workspace_bytes(T, d_in, [W.shape[1] for W in Ws], R),
                                dtype=torch.uint8, device=X.device)
    arr = (CProjection * n)()
    for j in range(n):
        arr[j] = CProjection(_p(Ws[j]), Ws[j].stride(0), _p(As[j]) if R else None, As[j].stride(0) if R else 0,
                             _p(Bs[j]) if R else None, Bs[j].stride(0) if R else 0, _p(Ys[j]), Ys[j].stride(0),
                             Ws[j].shape[1])
    ct = table.c_struct() if table is not None else CChunkTable(None, None, None, None, None, None, 0)
    _check("cwl_apply_grouped", lib().cwl_apply_grouped(_p(X), X.stride(0), arr, n, T, d_in, R, ct, int(window),
                                                        _p(workspace), workspace.numel(), _p(status_word),
                                                        _stream_ptr(stream)))
    return Ys


def cwl_stream_state_bytes(n_seq: int, min_len: int) -> int:
    return int(lib().cwl_stream_state_bytes(n_seq, min_len))


class DeviceStream:
    """Device-resident decode-time scheduler state of n_seq sequences plus the row-gate buffer it fills."""

    def __init__(self, n_seq: int, policy: CPolicy, device="cuda"):
        self.n_seq, self.policy = int(n_seq), policy
        self.state = torch.empty(max(cwl_stream_state_bytes(n_seq, int(policy.min_len)), 16), dtype=torch.uint8, device=device)
        self.gates = torch.zeros(max(n_seq, 1), ROW_GATE_BYTES, dtype=torch.uint8, device=device)
        self.reset()

    def reset(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        _check("cwl_stream_reset", lib().cwl_stream_reset(_p(self.state), self.state.numel(), self.n_seq,
                                                          int(self.policy.min_len), _stream_ptr(stream)))

    def step(self, score: torch.Tensor, active: Optional[torch.Tensor] = None,
             stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """Advances every (active) sequence by one token; returns the gate buffer ([n_seq, 28] bytes on the device)."""
        assert score.is_cuda and score.dtype == torch.float32 and score.is_contiguous() and score.numel() == self.n_seq
        if active is not None:
            assert active.is_cuda and active.dtype == torch.int32 and active.is_contiguous()
        _check("cwl_stream_step", lib().cwl_stream_step(_p(score), _p(active), self.n_seq, C.byref(self.policy),
                                                        _p(self.state), self.state.numel(), _p(self.gates),
                                                        _stream_ptr(stream)))
        return self.gates

    def gates_to_host(self):
        import numpy as np
        dt = np.dtype([("rank_in", np.int32), ("rank_out", np.int32), ("scale_in", np.float32), ("scale_out", np.float32),
                       ("lam", np.float32), ("pos_in_chunk", np.int32), ("opened", np.int32)])
        return self.gates[:self.n_seq].cpu().numpy().view(dt).reshape(self.n_seq)


def cwl_apply_rows(X: torch.Tensor, W: torch.Tensor, A: torch.Tensor, B: torch.Tensor, gates: torch.Tensor,
                   Y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                   status_word: Optional[torch.Tensor] = None,
                   stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """cwl_apply with one (rank, scale, lambda) descriptor per row; ``gates`` is a [T, 28]-byte device tensor."""
    T, d_in = X.shape
    d_out, R = W.shape[1], A.shape[1]
    assert gates.is_cuda and gates.dtype == torch.uint8 and gates.is_contiguous() and gates.numel() >= T * ROW_GATE_BYTES
    if Y is None:
        Y = torch.empty(T, d_out, dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = torch.empty(cwl_apply_workspace_bytes(T, d_in, d_out, R), dtype=torch.uint8, device=X.device)
    _check("cwl_apply_rows", lib().cwl_apply_rows(_p(X), X.stride(0), _p(W), W.stride(0), _p(A), A.stride(0),
                                                  _p(B), B.stride(0), T, d_in, d_out, R, _p(gates), _p(Y), Y.stride(0),
                                                  _p(workspace), workspace.numel(), _p(status_word), _stream_ptr(stream)))
    return Y


def cwl_ladder_build(A: torch.Tensor, B: torch.Tensor, want_f32: bool = True,
                     stream: Optional[torch.cuda.Stream] = None) -> dict:
    """SVD-ordered adapter factors of a trained (A [d_in, R], B [R, d_out]) pair, bf16 on the device (offline).
    Returns dict(A=bf16, B=bf16, sigma=fp32[R], sweeps=int) and, with want_f32, A32 / B32."""
    assert A.is_cuda and B.is_cuda and A.dtype == torch.bfloat16 and B.dtype == torch.bfloat16
    assert A.stride(1) == 1 and B.stride(1) == 1
    d_in, R = A.shape
    d_out = B.shape[1]
    out = dict(A=torch.empty(d_in, R, dtype=torch.bfloat16, device=A.device),
               B=torch.empty(R, d_out, dtype=torch.bfloat16, device=A.device),
               sigma=torch.empty(R, dtype=torch.float32, device=A.device))
    if want_f32:
        out["A32"] = torch.empty(d_in, R, dtype=torch.float32, device=A.device)
        out["B32"] = torch.empty(R, d_out, dtype=torch.float32, device=A.device)
    ws = torch.empty(max(int(lib().cwl_ladder_workspace_bytes(d_in, d_out, R)), 256), dtype=torch.uint8, device=A.device)
    sweeps = C.c_int32(0)
    _check("cwl_ladder_build", lib().cwl_ladder_build(
        _p(A), A.stride(0), _p(B), B.stride(0), d_in, d_out, R, _p(out["A"]), R, _p(out["B"]), d_out,
        _p(out.get("A32")), _p(out.get("B32")), _p(out["sigma"]), _p(ws), ws.numel(), C.byref(sweeps), _stream_ptr(stream)))
    out["sweeps"] = int(sweeps.value)
    return out


def cwl_apply_batch_workspace_bytes(T: int, d_ins: Sequence[int], d_outs: Sequence[int], R: int) -> int:
    n = len(d_ins)
    a = (C.c_int32 * n)(*[int(d) for d in d_ins])
    b = (C.c_int32 * n)(*[int(d) for d in d_outs])
    return int(lib().cwl_apply_batch_workspace_bytes(T, n, a, b, R))


class BatchCall:
    """A batch of independent projections with everything marshalled once: the item descriptors are built at
    construction, so a call costs one foreign call (decode steps are short enough for marshalling to show)."""

    def __init__(self, Xs: Sequence[torch.Tensor], Ws: Sequence[torch.Tensor], As: Optional[Sequence[torch.Tensor]],
                 Bs: Optional[Sequence[torch.Tensor]], Ys: Sequence[torch.Tensor], workspace: Optional[torch.Tensor] = None):
        n = len(Ws)
        self.T = int(Xs[0].shape[0])
        self.R = int(As[0].shape[1]) if As is not None else 0
        self.items = (CBatchItem * n)()
        for j in range(n):
            X, W, Y = Xs[j], Ws[j], Ys[j]
            assert X.dtype == torch.bfloat16 and W.dtype == torch.bfloat16 and X.shape[0] == self.T
            A = As[j] if As is not None else None
            B = Bs[j] if Bs is not None else None
            self.items[j] = CBatchItem(_p(X), X.stride(0), X.shape[1], _p(W), W.stride(0), _p(A), A.stride(0) if A is not None else 0,
                                       _p(B), B.stride(0) if B is not None else 0, _p(Y), Y.stride(0), W.shape[1])
        self.n = n
        self.keep = (list(Xs), list(Ws), list(As or []), list(Bs or []), list(Ys))
        need = cwl_apply_batch_workspace_bytes(self.T, [int(x.shape[1]) for x in Xs], [int(w.shape[1]) for w in Ws], self.R)
        self.workspace = workspace if workspace is not None else torch.empty(need, dtype=torch.uint8, device=Ws[0].device)
        assert self.workspace.numel() >= need

    def __call__(self, table: Optional["DeviceChunkTable"], window: int, gates: Optional[torch.Tensor] = None,
                 status_word: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> None:
        ct = table.c_struct() if table is not None else CChunkTable(None, None, None, None, None, None, 0)
        _check("cwl_apply_batch", lib().cwl_apply_batch(self.items, self.n, self.T, self.R, ct, _p(gates), int(window),
                                                        _p(self.workspace), self.workspace.numel(), _p(status_word),
                                                        _stream_ptr(stream)))


def cwl_set_pair_budget(pairs: int) -> None:
    """Apply calls of this thread plan for at most `pairs` CTA pairs from now on (0: the whole GPU)."""
    _check("cwl_set_pair_budget", lib().cwl_set_pair_budget(int(pairs)))


def cwl_prefetch_next(t: Optional[torch.Tensor], max_bytes: Optional[int] = None) -> None:
    """One-shot hint: the next apply call of this thread asks L2, while it drains, for the memory of `t` (the
    weights the call after it will stream), or for its first `max_bytes` bytes.  None withdraws a pending hint."""
    if t is None:
        lib().cwl_prefetch_next(None, 0)
    else:
        n = t.numel() * t.element_size()
        _check("cwl_prefetch_next", lib().cwl_prefetch_next(_p(t), n if max_bytes is None else min(n, int(max_bytes))))


def cwl_debug_set(wait_limit_ns: int = 0, withhold_publish: bool = False) -> None:
    """Test hook, inside ``with test_hooks():`` only: device-side wait limit (<= 0: default) and whether the shrink
    withholds H' (timeout path)."""
    if _lib is not _hooks_lib or _hooks_lib is None:
        raise RuntimeError("cwl_debug_set exists in the test build only: call it inside `with binding.test_hooks():`")
    _hooks_lib.cwl_debug_set(int(wait_limit_ns), 1 if withhold_publish else 0)


def cwl_apply_noalloc(X: torch.Tensor, W: torch.Tensor, A: Optional[torch.Tensor], B: Optional[torch.Tensor],
                      table: Optional[DeviceChunkTable], window: int, Y: torch.Tensor,
                      status_word: Optional[torch.Tensor] = None,
                      stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """cwl_apply for callers that cannot allocate on the device: no workspace argument, the scratch
    is the library's own fixed array (NOALLOC_SCRATCH_BYTES).  ``Y`` must be supplied by the caller;
    this wrapper creates no tensor.  Calls that overlap on the GPU race on the shared scratch."""
    T, d_in = X.shape
    d_out = W.shape[1]
    R = A.shape[1] if (A is not None and B is not None) else 0
    ct = table.c_struct() if table is not None else CChunkTable(None, None, None, None, None, None, 0)
    _check("cwl_apply_noalloc", lib().cwl_apply_noalloc(
        _p(X), X.stride(0), _p(W), W.stride(0), _p(A), A.stride(0) if R else 0, _p(B), B.stride(0) if R else 0,
        T, d_in, d_out, R, ct, int(window), _p(Y), Y.stride(0), _p(status_word), _stream_ptr(stream)))
    return Y


def bf16_from_bits(bits, device="cuda") -> torch.Tensor:
    """uint16 bit patterns (numpy) -> bf16 tensor on the device, no rounding involved."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)
