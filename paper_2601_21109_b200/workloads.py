"""Seeded synthetic inputs for the five benchmark configurations.

This module holds NO arithmetic of the method: it only draws random tensors with the shapes,
value distributions and structure of the workloads (LLaMA-7B projection sizes 4096/11008,
vocabulary 32000, ragged packed batches) and rounds them to their storage type once.  The same
host arrays are handed to the CUDA library and to the CPU oracle, so a comparison measures kernel
arithmetic and not input rounding.  Nothing here stands for the paper's datasets themselves
(Wikitext-103, SQuAD v2.0, FLORES-101 on LLaMA-7B, Sec. V-A): only their shapes are kept.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

SEED_BASE = 21109 * 10

# LLaMA-7B projection shapes (d_in, d_out)
LLAMA7B_PROJ: List[Tuple[str, int, int]] = [
    ("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
    ("gate", 4096, 11008), ("up", 4096, 11008), ("down", 11008, 4096),
]


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    """N(0, std^2) drawn in fp32, stored as bf16 bits."""
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))


@dataclass
class Policy:
    """Chunker / selector settings (the paper names them in Sec. III-B and III-C, gives no values)."""
    ranks: List[int]
    scales: List[float]
    thresholds: List[float]
    min_len: int
    max_len: int
    window: int
    hi_budget: int = -1

    @staticmethod
    def ladder(ranks: List[int], alpha: float, thresholds: List[float], min_len: int,
               window: int, max_len: Optional[int] = None, hi_budget: int = -1) -> "Policy":
        scales = [float(np.float32(alpha / r)) if r > 0 else 0.0 for r in ranks]
        return Policy(list(ranks), scales, [float(np.float32(t)) for t in thresholds], min_len,
                      max_len if max_len is not None else 16 * min_len, window, hi_budget)


@dataclass
class Projection:
    name: str
    d_in: int
    d_out: int
    W: np.ndarray  # bf16 bits [d_in, d_out]
    A: np.ndarray  # bf16 bits [d_in, R]
    B: np.ndarray  # bf16 bits [R, d_out]


@dataclass
class Workload:
    name: str
    T: int
    R: int
    policy: Policy
    cu_seqlens: np.ndarray                       # int32 [n_seq+1]
    X: Dict[int, np.ndarray]                     # d_in -> bf16 bits [T, d_in]
    projections: List[Projection]
    score: Optional[np.ndarray] = None           # fp32 [T] when scores are given
    logits: Optional[np.ndarray] = None          # fp32 [T, V] when scores come from logits
    table: Optional[dict] = None                 # explicit chunk table (decode config)
    notes: dict = field(default_factory=dict)


def make_projection(rng, name: str, d_in: int, d_out: int, R: int, b_std: Optional[float] = None) -> Projection:
    W = normal_bf16(rng, (d_in, d_out), d_in ** -0.5)
    A = normal_bf16(rng, (d_in, R), d_in ** -0.5)
    B = normal_bf16(rng, (R, d_out), b_std if b_std is not None else R ** -0.5)
    return Projection(name, d_in, d_out, W, A, B)


def span_temperature_logits(rng, T: int, V: int, span: int = 64) -> np.ndarray:
    """fp32 logits g / tau with g ~ N(0,1) and one tau ~ U[0.3, 3] per `span` tokens."""
    n_span = (T + span - 1) // span
    tau = rng.uniform(0.3, 3.0, size=n_span).astype(np.float32)
    z = rng.standard_normal((T, V), dtype=np.float32)
    z /= np.repeat(tau, span)[:T, None]
    return z


def config1(seed: int = SEED_BASE + 1) -> Workload:
    """Single 1024x1024 projection, T = 256, R = 16, ladder {4, 8, 16}, planted hard spans."""
    rng = np.random.default_rng(seed)
    T, d, R = 256, 1024, 16
    X = normal_bf16(rng, (T, d), 1.0)
    proj = make_projection(rng, "p", d, d, R, b_std=0.25)  # B ~ N(0, 1/16)
    score = rng.uniform(0.0, 1.0, size=T).astype(np.float32)
    # three non-overlapping 24-token spans of high scores, >= 16 apart, >= 8 from the ends
    starts: List[int] = []
    while len(starts) < 3:
        s = int(rng.integers(8, T - 8 - 24 + 1))
        if all(abs(s - o) >= 24 + 16 for o in starts):
            starts.append(s)
    for s in starts:
        score[s:s + 24] = rng.uniform(0.8, 1.0, size=24).astype(np.float32)
    score = np.minimum(score, np.float32(np.nextafter(np.float32(1.0), np.float32(0.0))))
    pol = Policy.ladder([4, 8, 16], 16.0, [0.33, 0.66], min_len=8, window=4)
    return Workload("cfg1_single_1024", T, R, pol, np.array([0, T], np.int32), {d: X}, [proj],
                    score=score, notes={"planted_starts": sorted(starts)})


def config2(seed: int = SEED_BASE + 2, T: int = 2048, V: int = 32000,
            projections: Optional[List[Tuple[str, int, int]]] = None,
            with_logits: bool = True) -> Workload:
    """LLaMA-7B-shaped single-sequence prefill: 7 projections, R = 64, ladder {8,16,32,64}.

    Thresholds are left empty: the harness fills them with the 25/50/75-th percentiles of the
    score array it partitions (the rule-based percentile mapping of Sec. IV-C)."""
    rng = np.random.default_rng(seed)
    R = 64
    logits = span_temperature_logits(rng, T, V) if with_logits else None
    plist = projections if projections is not None else LLAMA7B_PROJ
    X = {d: normal_bf16(rng, (T, d), 1.0) for d in sorted({p[1] for p in plist})}
    projs = [make_projection(rng, n, di, do, R) for (n, di, do) in plist]
    pol = Policy.ladder([8, 16, 32, 64], 32.0, [0.25, 0.5, 0.75], min_len=16, window=8)
    return Workload("cfg2_llama7b_prefill", T, R, pol, np.array([0, T], np.int32), X, projs, logits=logits)


def markov_scores(rng, lengths: np.ndarray, switch_p: float = 1.0 / 48.0) -> np.ndarray:
    """Two-regime (easy/hard) score track per sequence, restarted at each sequence."""
    out = []
    for L in lengths:
        L = int(L)
        s = np.empty(L, dtype=np.float64)
        hard = bool(rng.integers(0, 2))
        level = (0.75 if hard else 0.25) + rng.uniform(-0.2, 0.2)
        flips = rng.random(L) < switch_p
        for t in range(L):
            if t > 0 and flips[t]:
                hard = not hard
                level = (0.75 if hard else 0.25) + rng.uniform(-0.2, 0.2)
            s[t] = level
        s += rng.normal(0.0, 0.05, size=L)
        out.append(s)
    s = np.concatenate(out) if out else np.zeros(0)
    hi = np.nextafter(np.float32(1.0), np.float32(0.0))
    return np.clip(s, 0.0, hi).astype(np.float32)


def config3(seed: int = SEED_BASE + 3, n_seq: int = 32, d: int = 4096) -> Workload:
    """Packed ragged prefill: lognormal lengths (median 1024, clipped to 128..4096)."""
    rng = np.random.default_rng(seed)
    R = 64
    lengths = np.clip(np.rint(np.exp(rng.normal(np.log(1024.0), 0.6, size=n_seq))), 128, 4096).astype(np.int64)
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    T = int(cu[-1])
    score = markov_scores(rng, lengths)
    X = normal_bf16(rng, (T, d), 1.0)
    proj = make_projection(rng, "p", d, d, R)
    pol = Policy.ladder([4, 8, 16, 32, 64], 32.0, [0.2, 0.4, 0.6, 0.8], min_len=16, window=8)
    return Workload("cfg3_packed_ragged", T, R, pol, cu, {d: X}, [proj], score=score,
                    notes={"lengths": lengths.tolist()})


def config4(seed: int = SEED_BASE + 4, T: int = 256) -> Workload:
    """Decode step: T independent one-token sequences, each row with its own ladder rank."""
    rng = np.random.default_rng(seed)
    R = 64
    ladder = np.array([8, 16, 32, 64], dtype=np.int32)
    rung = rng.integers(0, 4, size=T).astype(np.int32)
    rank = ladder[rung]
    table = dict(offsets=np.arange(T + 1, dtype=np.int32), rank=rank.astype(np.int32),
                 scale=(np.float32(32.0) / rank.astype(np.float32)).astype(np.float32),
                 rung=rung, flags=np.ones(T, dtype=np.int32), n_chunks=T)
    X = {4096: normal_bf16(rng, (T, 4096), 1.0), 11008: normal_bf16(rng, (T, 11008), 1.0)}
    projs = [make_projection(rng, "up", 4096, 11008, R), make_projection(rng, "down", 11008, 4096, R)]
    pol = Policy.ladder([8, 16, 32, 64], 32.0, [0.25, 0.5, 0.75], min_len=1, window=0, max_len=1)
    return Workload("cfg4_decode", T, R, pol, np.arange(T + 1, dtype=np.int32), X, projs, table=table)


def config5_layer(seed: int = SEED_BASE + 5, n_seq: int = 4, seq_len: int = 4096, V: int = 32000,
                  with_logits: bool = True) -> Workload:
    """One layer of the 32-layer projection stack: 4 x 4096 tokens, 7 projections, R = 64.

    Every layer reads the same activations and logits; layers differ in their weights only, so
    a stack is this layer repeated with per-layer weight sets."""
    rng = np.random.default_rng(seed)
    T = n_seq * seq_len
    w = config2(seed=int(rng.integers(1 << 31)), T=T, V=V, with_logits=with_logits)
    w.name = "cfg5_stack_layer"
    w.cu_seqlens = (np.arange(n_seq + 1) * seq_len).astype(np.int32)
    return w


def static_table(cu_seqlens: np.ndarray, R: int, alpha: float) -> dict:
    """Chunk table of static full-rank LoRA: one chunk per (non-empty) sequence, rank R, scale alpha/R."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    keep = np.nonzero(np.diff(cu) > 0)[0]
    offsets = np.concatenate([cu[keep], cu[-1:]]).astype(np.int32)
    n = len(keep)
    return dict(offsets=offsets, rank=np.full(n, R, np.int32), scale=np.full(n, alpha / R, np.float32),
                rung=np.zeros(n, np.int32), flags=np.ones(n, np.int32), n_chunks=n)


def sample_rows(rng, T: int, offsets: np.ndarray, flags: np.ndarray, window: int,
                n_random: int = 64, n_joins: int = 8, n_chunks_edges: int = 8) -> np.ndarray:
    """Rows on which a large configuration is compared one by one: random rows, every window row
    of a few joins, first/last rows of a few chunks, and the first and last row overall."""
    rows = {0, T - 1}
    rows.update(int(r) for r in rng.integers(0, T, size=min(n_random, T)))
    C = len(offsets) - 1
    joins = [c for c in range(1, C) if not (flags[c] & 1)]
    for c in (rng.choice(joins, size=min(n_joins, len(joins)), replace=False) if joins else []):
        o = int(offsets[c])
        rows.update(range(max(0, o - 1), min(T, o + window + 1)))
    for c in rng.choice(C, size=min(n_chunks_edges, C), replace=False):
        rows.add(int(offsets[c]))
        rows.add(int(offsets[c + 1]) - 1)
    return np.array(sorted(r for r in rows if 0 <= r < T), dtype=np.int32)
