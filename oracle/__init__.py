"""fp64 CPU oracle of the ChunkWise-LoRA hot path -- TEST INFRASTRUCTURE ONLY.

A thin ctypes/numpy front for ``cwlo.c`` (plain C, fp64, naive loops).  It is independent of the
CUDA library: it imports nothing from the product package and the product never imports it.  Only
the test-suite, the smoke check and the benchmark's CPU-baseline leg may use it.

Functions follow the paper's sections: ``score_tokens`` (Sec. III-A signal (i)), ``partition``
(Sec. III-B chunker + Sec. III-C selector), ``blend_weights`` (Sec. III-D) and ``apply``
(Sec. III-F adapted projection with the cross-fade of Sec. III-D).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cwlo.c")
_HDR = os.path.join(_HERE, "cwlo.h")
_LIB = os.path.join(_HERE, "libcwlo.so")
MAX_RUNGS = 8


def build(force: bool = False) -> str:
    """Compile cwlo.c with gcc into libcwlo.so (rebuilt when a source is newer)."""
    stale = (not os.path.exists(_LIB)
             or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-fno-fast-math",
               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


class _Policy(C.Structure):
    _fields_ = [("n_rungs", C.c_int32),
                ("rung_rank", C.c_int32 * MAX_RUNGS),
                ("rung_scale", C.c_float * MAX_RUNGS),
                ("threshold", C.c_float * (MAX_RUNGS - 1)),
                ("min_len", C.c_int32), ("max_len", C.c_int32),
                ("window", C.c_int32), ("hi_budget", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.cwlo_quantise.restype = C.c_int64
        _lib.cwlo_quantise.argtypes = [C.c_float]
        _lib.cwlo_rung.restype = C.c_int32
        _lib.cwlo_rung.argtypes = [C.c_int64, C.c_int64, C.POINTER(_Policy)]
        _lib.cwlo_blend_weight.restype = C.c_double
        _lib.cwlo_blend_weight_centred.restype = C.c_double
        _lib.cwlo_get_threads.restype = C.c_int
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _policy_struct(ranks: Sequence[int], scales: Sequence[float], thresholds: Sequence[float],
                   min_len: int, max_len: int, window: int, hi_budget: int) -> _Policy:
    p = _Policy()
    p.n_rungs = len(ranks)
    for k, r in enumerate(ranks):
        p.rung_rank[k] = int(r)
    for k, s in enumerate(scales):
        p.rung_scale[k] = float(s)
    for k, th in enumerate(thresholds):
        p.threshold[k] = float(th)
    p.min_len, p.max_len, p.window, p.hi_budget = int(min_len), int(max_len), int(window), int(hi_budget)
    return p


@dataclass
class ChunkTable:
    offsets: np.ndarray  # int32 [C+1]
    rank: np.ndarray     # int32 [C]
    scale: np.ndarray    # float32 [C]
    rung: np.ndarray     # int32 [C]
    flags: np.ndarray    # int32 [C], bit0 = first chunk of its sequence
    n_chunks: int = field(default=0)


def get_threads() -> int:
    return int(lib().cwlo_get_threads())


def set_threads(n: int) -> None:
    lib().cwlo_set_threads(C.c_int(int(n)))


def score_tokens(logits: np.ndarray) -> np.ndarray:
    """Normalised softmax entropy per row of fp32 ``logits`` [T, V]; returns fp64 [T]."""
    z = np.ascontiguousarray(logits, dtype=np.float32)
    T, V = z.shape
    out = np.empty(T, dtype=np.float64)
    rc = lib().cwlo_score_tokens(_ptr(z), C.c_int64(V), C.c_int32(T), C.c_int32(V), _ptr(out))
    if rc != 0:
        raise ValueError(f"cwlo_score_tokens: status {rc}")
    return out


def quantise(s: float) -> int:
    return int(lib().cwlo_quantise(C.c_float(float(s))))


def rung_of(total: int, length: int, ranks, scales, thresholds, min_len=1, max_len=1) -> int:
    p = _policy_struct(ranks, scales, thresholds, min_len, max_len, 0, -1)
    return int(lib().cwlo_rung(C.c_int64(int(total)), C.c_int64(int(length)), C.byref(p)))


def partition(score: np.ndarray, cu_seqlens: np.ndarray, ranks, scales, thresholds,
              min_len: int, max_len: int, window: int = 0, hi_budget: int = -1,
              capacity: Optional[int] = None) -> ChunkTable:
    """Adaptive chunker + rank-ladder selector on an fp32 score array."""
    s = np.ascontiguousarray(score, dtype=np.float32)
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    T, n_seq = s.shape[0], cu.shape[0] - 1
    cap = int(capacity) if capacity is not None else T + n_seq + 1
    offsets = np.zeros(cap + 1, dtype=np.int32)
    rank = np.zeros(cap, dtype=np.int32)
    scale = np.zeros(cap, dtype=np.float32)
    rung = np.zeros(cap, dtype=np.int32)
    flags = np.zeros(cap, dtype=np.int32)
    n = C.c_int32(0)
    p = _policy_struct(ranks, scales, thresholds, min_len, max_len, window, hi_budget)
    rc = lib().cwlo_partition(_ptr(s), _ptr(cu), C.c_int32(n_seq), C.c_int32(T), C.byref(p),
                              _ptr(offsets), _ptr(rank), _ptr(scale), _ptr(rung), _ptr(flags),
                              C.byref(n), C.c_int32(cap))
    if rc == 4:
        raise OverflowError("cwlo_partition: chunk table capacity exceeded")
    if rc != 0:
        raise ValueError(f"cwlo_partition: status {rc}")
    c = n.value
    return ChunkTable(offsets[:c + 1].copy(), rank[:c].copy(), scale[:c].copy(), rung[:c].copy(),
                      flags[:c].copy(), c)


def batch_align(score: np.ndarray, cu_seqlens: np.ndarray, ranks, scales, thresholds, min_len: int, max_len: int,
                n_buckets: int, window: int = 0, hi_budget: int = -1, capacity: Optional[int] = None):
    """Batch alignment: sequences bucketed by complexity percentile share their chunk joins.
    Returns (ChunkTable, bucket [n_seq], order_pos [n_seq])."""
    s = np.ascontiguousarray(score, dtype=np.float32)
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    T, n_seq = s.shape[0], cu.shape[0] - 1
    cap = int(capacity) if capacity is not None else T + n_seq + 1
    offsets = np.zeros(cap + 1, dtype=np.int32)
    rank = np.zeros(cap, dtype=np.int32)
    scale = np.zeros(cap, dtype=np.float32)
    rung = np.zeros(cap, dtype=np.int32)
    flags = np.zeros(cap, dtype=np.int32)
    bucket = np.zeros(max(n_seq, 1), dtype=np.int32)
    order_pos = np.zeros(max(n_seq, 1), dtype=np.int32)
    n = C.c_int32(0)
    p = _policy_struct(ranks, scales, thresholds, min_len, max_len, window, hi_budget)
    rc = lib().cwlo_batch_align(_ptr(s), _ptr(cu), C.c_int32(n_seq), C.c_int32(T), C.byref(p), C.c_int32(n_buckets),
                                _ptr(offsets), _ptr(rank), _ptr(scale), _ptr(rung), _ptr(flags),
                                C.byref(n), C.c_int32(cap), _ptr(bucket), _ptr(order_pos))
    if rc == 4:
        raise OverflowError("cwlo_batch_align: chunk table capacity exceeded")
    if rc != 0:
        raise ValueError(f"cwlo_batch_align: status {rc}")
    c = n.value
    tab = ChunkTable(offsets[:c + 1].copy(), rank[:c].copy(), scale[:c].copy(), rung[:c].copy(), flags[:c].copy(), c)
    return tab, bucket[:n_seq].copy(), order_pos[:n_seq].copy()


def blend_weights(table: ChunkTable, T: int, window: int) -> np.ndarray:
    """Weight of the incoming configuration for every row (fp64 [T])."""
    off = np.ascontiguousarray(table.offsets, dtype=np.int32)
    fl = np.ascontiguousarray(table.flags, dtype=np.int32)
    out = np.empty(T, dtype=np.float64)
    f = lib().cwlo_blend_weight
    for t in range(T):
        out[t] = f(C.c_int32(t), _ptr(off), _ptr(fl), C.c_int32(table.n_chunks), C.c_int32(window), None)
    return out


def blend_weights_centred(table: ChunkTable, T: int, window: int):
    """Centred window placement: (weight of cfg_in, cfg_in, cfg_out) for every row."""
    off = np.ascontiguousarray(table.offsets, dtype=np.int32)
    fl = np.ascontiguousarray(table.flags, dtype=np.int32)
    lam = np.empty(T, dtype=np.float64)
    cin = np.empty(T, dtype=np.int32)
    cout = np.empty(T, dtype=np.int32)
    f = lib().cwlo_blend_weight_centred
    a, b = C.c_int32(0), C.c_int32(0)
    for t in range(T):
        lam[t] = f(C.c_int32(t), _ptr(off), _ptr(fl), C.c_int32(table.n_chunks), C.c_int32(window), C.byref(a), C.byref(b))
        cin[t], cout[t] = a.value, b.value
    return lam, cin, cout


def apply(X: np.ndarray, W: np.ndarray, A: Optional[np.ndarray], B: Optional[np.ndarray],
          table: Optional[ChunkTable], window: int, rows: Optional[np.ndarray] = None,
          centred: bool = False) -> np.ndarray:
    """Adapted projection in fp64.  X, W, A, B are uint16 arrays of bf16 bit patterns.
    ``centred`` places the cross-fade window around each join instead of after it.

    Returns Y [T, d_out] or, with ``rows``, Y [len(rows), d_out] in list order."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    W = np.ascontiguousarray(W, dtype=np.uint16)
    T, d_in = X.shape
    d_out = W.shape[1]
    assert W.shape[0] == d_in
    R = 0
    if A is not None and B is not None:
        A = np.ascontiguousarray(A, dtype=np.uint16)
        B = np.ascontiguousarray(B, dtype=np.uint16)
        R = A.shape[1]
        assert A.shape[0] == d_in and B.shape == (R, d_out)
    else:
        A = B = None
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int32)
        n_rows = rows.shape[0]
    else:
        n_rows = T
    Y = np.empty((n_rows, d_out), dtype=np.float64)
    if table is not None:
        off = np.ascontiguousarray(table.offsets, dtype=np.int32)
        rk = np.ascontiguousarray(table.rank, dtype=np.int32)
        sc = np.ascontiguousarray(table.scale, dtype=np.float32)
        fl = np.ascontiguousarray(table.flags, dtype=np.int32)
        nc = int(table.n_chunks)
    else:
        off = rk = sc = fl = None
        nc = 0
    fn = lib().cwlo_apply_centred if centred else lib().cwlo_apply
    rc = fn(_ptr(X), C.c_int64(d_in), _ptr(W), C.c_int64(d_out),
                          _ptr(A), C.c_int64(R), _ptr(B), C.c_int64(d_out),
                          C.c_int32(T), C.c_int32(d_in), C.c_int32(d_out), C.c_int32(R),
                          _ptr(off), _ptr(rk), _ptr(sc), _ptr(fl), C.c_int32(nc), C.c_int32(window),
                          _ptr(rows), C.c_int32(n_rows), _ptr(Y), C.c_int64(d_out))
    if rc != 0:
        raise ValueError(f"cwlo_apply: status {rc}")
    return Y


# ------------------------------------------------------------------ decode-time scheduler (streaming)
STREAM_MAX_MIN_LEN = 64


class _StreamState(C.Structure):
    _fields_ = [("pos", C.c_int32), ("len", C.c_int32), ("cur_rung", C.c_int32), ("prev_rung", C.c_int32),
                ("hi_used", C.c_int32), ("first", C.c_int32), ("ring", C.c_int64 * STREAM_MAX_MIN_LEN)]


class RowGate(C.Structure):
    _fields_ = [("rank_in", C.c_int32), ("rank_out", C.c_int32), ("scale_in", C.c_float), ("scale_out", C.c_float),
                ("lambda_", C.c_float), ("pos_in_chunk", C.c_int32), ("opened", C.c_int32)]


ROW_GATE_DTYPE = np.dtype([("rank_in", np.int32), ("rank_out", np.int32), ("scale_in", np.float32),
                           ("scale_out", np.float32), ("lam", np.float32), ("pos_in_chunk", np.int32),
                           ("opened", np.int32)])


class Stream:
    """Decode-time scheduler of ONE sequence (Sec. III-B: tokens are grouped as they arrive; the state is kept from step to step)."""

    def __init__(self, ranks, scales, thresholds, min_len, max_len, window, hi_budget=-1):
        self.policy = _policy_struct(ranks, scales, thresholds, min_len, max_len, window, hi_budget)
        self.state = _StreamState()
        lib().cwlo_stream_reset(C.byref(self.state))

    def step(self, score: float) -> np.void:
        g = RowGate()
        rc = lib().cwlo_stream_step(C.byref(self.state), C.c_float(float(score)), C.byref(self.policy), C.byref(g))
        if rc != 0:
            raise ValueError(f"cwlo_stream_step: status {rc}")
        out = np.zeros((), dtype=ROW_GATE_DTYPE)
        out["rank_in"], out["rank_out"], out["scale_in"], out["scale_out"] = g.rank_in, g.rank_out, g.scale_in, g.scale_out
        out["lam"], out["pos_in_chunk"], out["opened"] = g.lambda_, g.pos_in_chunk, g.opened
        return out


def apply_rows(X: np.ndarray, W: np.ndarray, A: np.ndarray, B: np.ndarray, gates: np.ndarray) -> np.ndarray:
    """Adapted projection in fp64 with one (rank_in, scale_in, rank_out, scale_out, lambda) descriptor per row.
    ``gates`` is a structured array of ROW_GATE_DTYPE."""
    X = np.ascontiguousarray(X, dtype=np.uint16); W = np.ascontiguousarray(W, dtype=np.uint16)
    A = np.ascontiguousarray(A, dtype=np.uint16); B = np.ascontiguousarray(B, dtype=np.uint16)
    gates = np.ascontiguousarray(gates, dtype=ROW_GATE_DTYPE)
    T, d_in = X.shape
    d_out, R = W.shape[1], A.shape[1]
    assert gates.shape == (T,) and ROW_GATE_DTYPE.itemsize == C.sizeof(RowGate)
    Y = np.empty((T, d_out), dtype=np.float64)
    rc = lib().cwlo_apply_rows(_ptr(X), C.c_int64(d_in), _ptr(W), C.c_int64(d_out), _ptr(A), C.c_int64(R),
                               _ptr(B), C.c_int64(d_out), C.c_int32(T), C.c_int32(d_in), C.c_int32(d_out), C.c_int32(R),
                               gates.ctypes.data_as(C.c_void_p), _ptr(Y), C.c_int64(d_out))
    if rc != 0:
        raise ValueError(f"cwlo_apply_rows: status {rc}")
    return Y


# ------------------------------------------------------------------ further complexity signals (Sec. III-A (ii), (iv))
class _SignalMix(C.Structure):
    _fields_ = [("w_entropy", C.c_float), ("w_novelty", C.c_float), ("w_prior", C.c_float),
                ("ngram", C.c_int32), ("context", C.c_int32), ("prior_span", C.c_int32)]


def score_tokens_mixed(logits: np.ndarray, token_ids: np.ndarray, cu_seqlens: np.ndarray, w_entropy: float,
                       w_novelty: float, w_prior: float, ngram: int, context: int, prior_span: int) -> np.ndarray:
    """clamp(w_e * entropy + w_n * n-gram novelty + w_p * positional prior, 0, 1) per token, fp64 [T]."""
    z = np.ascontiguousarray(logits, dtype=np.float32)
    ids = np.ascontiguousarray(token_ids, dtype=np.int32)
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    T, V = z.shape
    mix = _SignalMix(float(w_entropy), float(w_novelty), float(w_prior), int(ngram), int(context), int(prior_span))
    out = np.empty(T, dtype=np.float64)
    rc = lib().cwlo_score_tokens_mixed(_ptr(z), C.c_int64(V), C.c_int32(T), C.c_int32(V), _ptr(ids), _ptr(cu),
                                       C.c_int32(len(cu) - 1), C.byref(mix), _ptr(out))
    if rc != 0:
        raise ValueError(f"cwlo_score_tokens_mixed: status {rc}")
    return out


# ------------------------------------------------------------------ offline ladder construction (Sec. III-C)
def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def svd_ladder(A: np.ndarray, B: np.ndarray):
    """SVD-ordered adapter factors (Sec. III-C: the trained update is re-factorised once by SVD so that every
    prefix of the factors is a usable adapter).  A [d_in, R], B [R, d_out] are bf16 bit patterns.  With
    A B = U diag(sigma) V^T (singular values in descending order, numpy's LAPACK SVD as the library step) returns
    (A' = U diag(sigma) [d_in, R], B' = V^T [R, d_out], sigma [R]) in fp64, so that A'[:, :r] B'[:r, :] is the best
    rank-r approximation of A B for every r (Eckart-Young)."""
    a, b = _bf16_to_f64(A), _bf16_to_f64(B)
    R = a.shape[1]
    U, s, Vt = np.linalg.svd(a @ b, full_matrices=False)
    return U[:, :R] * s[:R], Vt[:R, :], s[:R]
