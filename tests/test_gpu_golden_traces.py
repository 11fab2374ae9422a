"""cwl_partition and cwl_stream_step on the hand-worked traces of tests/golden/ (the same files the
oracle is pinned with): the CUDA path must reproduce every cut, rung, demotion and gate of the trace itself,
not merely agree with the oracle."""
import os

import numpy as np
import pytest
import torch

from paper_2601_21109_b200 import binding as cwl
from test_oracle_golden_traces import GOLDEN, read_keyed

pytestmark = pytest.mark.gpu


def test_partition_trace_on_the_gpu():
    g = read_keyed(os.path.join(GOLDEN, "partition_tiny.txt"))
    score = torch.from_numpy((np.array(g["score_eighths"], np.float64) / 8.0).astype(np.float32)).cuda()
    cu = torch.from_numpy(np.array(g["cu_seqlens"], np.int32)).cuda()
    pol = cwl.make_policy([int(x) for x in g["ranks"]], [float(x) for x in g["scales"]], [float(x) for x in g["thresholds"]],
                          int(g["min_len"][0]), int(g["max_len"][0]), int(g["window"][0]), int(g["hi_budget"][0]))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = cwl.cwl_partition(score, cu, pol, status_word=status).to_host()
    assert int(status.item()) == 0
    n = len(g["rank"])
    assert got["n_chunks"] == n
    assert got["offsets"].tolist() == [int(x) for x in g["offsets"]]
    assert got["rung"].tolist() == [int(x) for x in g["rung"]]
    assert got["rank"].tolist() == [int(x) for x in g["rank"]]
    assert got["scale"].tolist() == [float(x) for x in g["scale"]]
    assert (got["flags"] & 1).tolist() == [int(x) for x in g["flags"]]


def test_stream_trace_on_the_gpu():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "stream_tiny.txt"))
            if l.strip() and not l.startswith("#") and not l.startswith("policy")]
    pol = cwl.make_policy([4, 8, 16], [4.0, 2.0, 1.0], [0.25, 0.75], 4, 8, 2, 1)
    ds = cwl.DeviceStream(2, pol)          # two sequences fed the same scores: both must follow the trace
    for t, eighths, opened, j, r_in, s_in, r_out, s_out, lam in rows:
        ds.step(torch.full((2,), int(eighths) / 8.0, dtype=torch.float32, device="cuda"))
        num, den = lam.split("/")
        want = (int(opened), int(j), int(r_in), float(s_in), int(r_out), float(s_out), np.float32(int(num)) / np.float32(int(den)))
        for g in ds.gates_to_host():
            got = (int(g["opened"]), int(g["pos_in_chunk"]), int(g["rank_in"]), float(g["scale_in"]), int(g["rank_out"]),
                   float(g["scale_out"]), np.float32(g["lam"]))
            assert got == want, f"token {t}: {got} != {want}"
