"""Pins of the oracle's decode-time scheduler (the causal, token-by-token chunker with cached state) and
of its per-row adapted projection.  The paper prints no rule for the online grouping (Sec. III-B names
the constraints only), so the rule is pinned internally: a run traced by hand, invariants that follow
from the constraints, and an independent brute force that rebuilds every decision from the whole score
history in exact integer arithmetic.  apply_rows is pinned against the (pinned) table-driven apply."""
import math

import numpy as np
import pytest

import oracle
from paper_2601_21109_b200 import workloads as wl

Q24 = 1 << 24
POL = dict(ranks=[4, 8, 16], scales=[4.0, 2.0, 1.0], thresholds=[0.33, 0.66])


def run_stream(scores, min_len, max_len, window, hi_budget=-1, pol=POL):
    s = oracle.Stream(pol["ranks"], pol["scales"], pol["thresholds"], min_len, max_len, window, hi_budget)
    return [s.step(x) for x in scores]


def test_hand_traced_run():
    # L_min = 2, L_max = 4, w = 1.  Five easy tokens: the first chunk is closed by the length cap at token 4;
    # the hard tokens from 5 on are seen by the two-token window at token 6, which opens a rank-16 chunk.
    out = run_stream([0.1] * 5 + [0.9] * 3, 2, 4, 1)
    got = [(int(g["opened"]), int(g["pos_in_chunk"]), int(g["rank_in"]), float(g["lam"]), int(g["rank_out"])) for g in out]
    assert got == [(1, 0, 4, 1.0, 0), (0, 1, 4, 1.0, 0), (0, 2, 4, 1.0, 0), (0, 3, 4, 1.0, 0),
                   (1, 0, 4, 0.5, 4), (0, 1, 4, 1.0, 0), (1, 0, 16, 0.5, 4), (0, 1, 16, 1.0, 0)]
    assert float(out[6]["scale_in"]) == 1.0 and float(out[6]["scale_out"]) == 4.0


def brute_force(scores, pol, min_len, max_len, window, hi_budget):
    """Every decision recomputed from the full history, integers only."""
    th = [math.floor(float(np.float32(t)) * Q24) for t in pol["thresholds"]]
    q = []
    for s in scores:
        s = float(np.float32(s))
        q.append(Q24 if math.isnan(s) else math.floor(min(max(s, 0.0), 1.0) * Q24))
    K = len(pol["ranks"])
    opens, rungs, top_flags, out = [], [], [], []      # where chunks opened, their rungs, whether they took a top-rung slot
    for t in range(len(q)):
        w = q[max(0, t - min_len + 1):t + 1]
        r_win = sum(1 for k in range(K - 1) if sum(w) >= th[k] * len(w))
        if t == 0:
            opened = True
        else:
            length = t - opens[-1]
            opened = length >= min_len and (length >= max_len or r_win != rungs[-1])
        if opened:
            if hi_budget >= 0 and K >= 2 and r_win == K - 1:
                if sum(top_flags) >= hi_budget:
                    r_win = K - 2
                    top_flags.append(0)
                else:
                    top_flags.append(1)
            else:
                top_flags.append(0)
            opens.append(t)
            rungs.append(r_win)
        j = t - opens[-1]
        lam, r_out = 1.0, 0
        if len(opens) > 1 and j < window:
            lam, r_out = float(np.float32(j + 1) / np.float32(window + 1)), pol["ranks"][rungs[-2]]
        out.append((int(opened), j, pol["ranks"][rungs[-1]], lam, r_out))
    return out


@pytest.mark.parametrize("seed", range(12))
def test_matches_brute_force_and_invariants(seed):
    rng = np.random.default_rng(100 + seed)
    min_len = int(rng.integers(1, 9))
    max_len = min_len * int(rng.integers(1, 6))
    window = int(rng.integers(0, min_len + 1))
    hi_budget = int(rng.choice([-1, 0, 1, 3]))
    n = 300
    # regimes with noise, so that rungs change; a few exact-threshold and out-of-range values
    level = np.repeat(rng.choice([0.1, 0.33, 0.5, 0.66, 0.9], size=n // 20 + 1), 20)[:n]
    scores = np.clip(level + rng.normal(0, 0.08, n), -0.2, 1.2).astype(np.float32)
    scores[rng.integers(0, n, 5)] = np.float32(0.33)
    out = run_stream(scores, min_len, max_len, window, hi_budget)
    got = [(int(g["opened"]), int(g["pos_in_chunk"]), int(g["rank_in"]), float(g["lam"]), int(g["rank_out"])) for g in out]
    assert got == brute_force(scores, POL, min_len, max_len, window, hi_budget)
    opens = [t for t, g in enumerate(got) if g[0]]
    lengths = np.diff(opens)
    assert opens[0] == 0 and (lengths >= min_len).all() and (lengths <= max_len).all()     # closed chunks respect both bounds
    assert n - opens[-1] <= max_len                                                      # so does the open one
    for t, g in enumerate(got):
        first = t < (opens[1] if len(opens) > 1 else n)
        if first or g[1] >= window:
            assert g[3] == 1.0 and g[4] == 0                                              # no blend outside a window
        else:
            assert g[3] == float(np.float32(g[1] + 1) / np.float32(window + 1))
    if hi_budget >= 0:
        assert sum(1 for t in opens if got[t][2] == POL["ranks"][-1]) <= hi_budget


def test_constant_scores_open_a_chunk_every_max_len_tokens():
    out = run_stream([0.5] * 50, 4, 12, 2)
    assert [t for t, g in enumerate(out) if g["opened"]] == [0, 12, 24, 36, 48]
    assert all(int(g["rank_in"]) == 8 for g in out)


def test_bad_policy_is_rejected():
    with pytest.raises(ValueError):
        run_stream([0.5], oracle.STREAM_MAX_MIN_LEN + 1, 2 * oracle.STREAM_MAX_MIN_LEN + 2, 0)


def test_apply_rows_equals_table_apply():
    rng = np.random.default_rng(5)
    T, d_in, d_out, R, w = 40, 32, 24, 16, 3
    X = wl.normal_bf16(rng, (T, d_in), 1.0); W = wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5)
    A = wl.normal_bf16(rng, (d_in, R), d_in ** -0.5); B = wl.normal_bf16(rng, (R, d_out), 0.25)
    offsets = np.array([0, 7, 15, 22, 40], np.int32)
    rank = np.array([4, 16, 0, 8], np.int32); scale = np.array([4.0, 1.0, 0.0, 2.0], np.float32)
    flags = np.array([1, 0, 1, 0], np.int32)
    tab = oracle.ChunkTable(offsets, rank, scale, np.zeros(4, np.int32), flags, 4)
    gates = np.zeros(T, dtype=oracle.ROW_GATE_DTYPE)
    for c in range(4):
        for t in range(offsets[c], offsets[c + 1]):
            j = t - offsets[c]
            gates[t]["rank_in"], gates[t]["scale_in"], gates[t]["lam"] = rank[c], scale[c], 1.0
            if not flags[c] & 1 and j < w:
                gates[t]["lam"] = np.float32(j + 1) / np.float32(w + 1)
                gates[t]["rank_out"], gates[t]["scale_out"] = rank[c - 1], scale[c - 1]
    y_rows = oracle.apply_rows(X, W, A, B, gates)
    y_tab = oracle.apply(X, W, A, B, tab, w)
    # the table path takes lambda in fp64, the row path reads it as fp32: equal to fp32 rounding of lambda
    assert np.max(np.abs(y_rows - y_tab)) <= 1e-6 * np.max(np.abs(y_tab))
    lam1 = gates["lam"] == 1.0
    assert np.array_equal(y_rows[lam1], y_tab[lam1])
