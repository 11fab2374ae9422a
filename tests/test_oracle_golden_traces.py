"""The chunker and the decode-time scheduler of the oracle against traces worked out by hand
(tests/golden/partition_tiny.txt, tests/golden/stream_tiny.txt).  The paper prints neither a rule nor an
example for either, so these traces pin the oracle to the documented reading of Sec. III-B / III-C / III-D,
decision by decision: cuts on a rung change, the length cap, the two tail rules, a budget tie, the
online budget, the cross-fade descriptors."""
import os

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_keyed(path):
    out = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        out[key] = vals
    return out


def test_partition_trace():
    g = read_keyed(os.path.join(GOLDEN, "partition_tiny.txt"))
    score = (np.array(g["score_eighths"], np.float64) / 8.0).astype(np.float32)
    cu = np.array(g["cu_seqlens"], np.int32)
    tab = oracle.partition(score, cu, [int(x) for x in g["ranks"]], [float(x) for x in g["scales"]],
                           [float(x) for x in g["thresholds"]], int(g["min_len"][0]), int(g["max_len"][0]),
                           int(g["window"][0]), int(g["hi_budget"][0]))
    n = len(g["rank"])
    assert tab.n_chunks == n
    assert tab.offsets[:n + 1].tolist() == [int(x) for x in g["offsets"]]
    assert tab.rung[:n].tolist() == [int(x) for x in g["rung"]]
    assert tab.rank[:n].tolist() == [int(x) for x in g["rank"]]
    assert tab.scale[:n].tolist() == [float(x) for x in g["scale"]]
    assert (tab.flags[:n] & 1).tolist() == [int(x) for x in g["flags"]]


def test_partition_trace_without_the_budget_keeps_both_top_rung_chunks():
    g = read_keyed(os.path.join(GOLDEN, "partition_tiny.txt"))
    score = (np.array(g["score_eighths"], np.float64) / 8.0).astype(np.float32)
    tab = oracle.partition(score, np.array(g["cu_seqlens"], np.int32), [4, 8, 16], [4.0, 2.0, 1.0], [0.25, 0.75], 4, 12, 2, -1)
    want = [int(x) for x in g["rung"]]
    want[7] = 2                                      # the chunk the budget demoted
    assert tab.rung[:tab.n_chunks].tolist() == want
    assert tab.offsets[:tab.n_chunks + 1].tolist() == [int(x) for x in g["offsets"]]   # the budget never moves a cut


def test_stream_trace():
    rows, pol = [], None
    for line in open(os.path.join(GOLDEN, "stream_tiny.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = line.split()
        if parts[0] == "policy":
            kv = {}
            key = None
            for p in parts[1:]:
                if p[0].isalpha():
                    key = p; kv[key] = []
                else:
                    kv[key].append(float(p))
            pol = kv
        else:
            rows.append(parts)
    s = oracle.Stream([int(x) for x in pol["ranks"]], pol["scales"], pol["thresholds"], int(pol["min_len"][0]),
                      int(pol["max_len"][0]), int(pol["window"][0]), int(pol["hi_budget"][0]))
    assert len(rows) == 40
    for t, eighths, opened, j, r_in, s_in, r_out, s_out, lam in rows:
        g = s.step(np.float32(int(eighths) / 8.0))
        num, den = lam.split("/")
        want_lam = np.float32(int(num)) / np.float32(int(den))
        got = (int(g["opened"]), int(g["pos_in_chunk"]), int(g["rank_in"]), float(g["scale_in"]), int(g["rank_out"]),
               float(g["scale_out"]), np.float32(g["lam"]))
        assert got == (int(opened), int(j), int(r_in), float(s_in), int(r_out), float(s_out), want_lam), f"token {t}: {got}"
