"""GPU parity of cwl_partition (chunker Sec. III-B + selector Sec. III-C): chunk offsets, ranks,
rungs, flags and scales must equal the oracle's bit for bit on the same fp32 scores."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run(score, cu, pol: wl.Policy, capacity=None):
    st = torch.from_numpy(np.ascontiguousarray(score, np.float32)).cuda()
    cut = torch.from_numpy(np.ascontiguousarray(cu, np.int32)).cuda()
    cp = cwl.make_policy(pol.ranks, pol.scales, pol.thresholds, pol.min_len, pol.max_len, pol.window, pol.hi_budget)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    table = None if capacity is None else cwl.DeviceChunkTable(capacity)
    tab = cwl.cwl_partition(st, cut, cp, table=table, status_word=status)
    torch.cuda.synchronize()
    return tab.to_host(), int(status.item())


def compare(score, cu, pol):
    got, status = run(score, cu, pol)
    assert status == 0
    ref = oracle.partition(score, cu, pol.ranks, pol.scales, pol.thresholds, pol.min_len, pol.max_len,
                           pol.window, pol.hi_budget)
    assert got["n_chunks"] == ref.n_chunks
    for key in ("offsets", "rank", "rung", "flags"):
        assert np.array_equal(got[key], getattr(ref, key)), key
    assert np.array_equal(got["scale"].view(np.uint32), ref.scale.view(np.uint32))
    return ref


def test_config1_scores():
    w = wl.config1()
    ref = compare(w.score, w.cu_seqlens, w.policy)
    assert ref.n_chunks <= 32


def test_config3_packed_ragged():
    w = wl.config3(d=16)
    ref = compare(w.score, w.cu_seqlens, w.policy)
    assert ref.n_chunks > 200


@pytest.mark.parametrize("seed", range(40))
def test_random_policies_and_scores(seed):
    rng = np.random.default_rng(5000 + seed)
    n_seq = int(rng.integers(1, 9))
    lens = rng.integers(0, 700, size=n_seq)
    if seed % 5 == 0:
        lens[rng.integers(0, n_seq)] = 0
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(cu[-1])
    kind = seed % 3
    if kind == 0:
        s = rng.random(T)
    elif kind == 1:
        s = np.repeat(rng.random(T // 7 + 1), 7)[:T] + rng.normal(0, 0.03, T)
    else:
        s = rng.integers(0, 5, T) / 4.0                       # exact ties at the thresholds
    s = s.astype(np.float32)
    if T and seed % 4 == 0:
        s[rng.integers(0, T, size=3)] = [np.nan, -0.5, 1.5]
    K = int(rng.integers(1, 6))
    ranks = sorted(rng.choice([0, 4, 8, 16, 32, 64], size=K, replace=False).tolist())
    ths = sorted(rng.choice([0.1, 0.25, 0.33, 0.5, 0.66, 0.75, 0.9], size=K - 1, replace=False).tolist())
    min_len = int(rng.integers(1, 20))
    pol = wl.Policy.ladder(ranks, 32.0, ths, min_len=min_len, window=0, max_len=min_len + int(rng.integers(0, 80)),
                           hi_budget=int(rng.choice([-1, 0, 1, 3])))
    compare(s, cu, pol)


def test_long_sequence_crosses_walk_segments():
    rng = np.random.default_rng(77)
    T = 40000
    s = (np.repeat(rng.random(T // 50 + 1), 50)[:T] + rng.normal(0, 0.02, T)).clip(0, 1).astype(np.float32)
    pol = wl.Policy.ladder([8, 16, 32, 64], 32.0, [0.25, 0.5, 0.75], min_len=16, window=8, hi_budget=5)
    compare(s, np.array([0, T], np.int32), pol)


@pytest.mark.parametrize("cu", [[0, 150000], [0, 70001, 70001, 149000, 150000]])
def test_more_than_32_scan_tiles(cu):
    """Above 65536 tokens the prefix sums take two passes (tile sums first); below, one.  Both sizes, with one
    sequence (the walk pass writes the table) and with several (the emit pass does), give the oracle's table."""
    rng = np.random.default_rng(78)
    T = cu[-1]
    s = (np.repeat(rng.random(T // 40 + 1), 40)[:T] + rng.normal(0, 0.03, T)).clip(0, 1).astype(np.float32)
    pol = wl.Policy.ladder([8, 16, 32, 64], 32.0, [0.25, 0.5, 0.75], min_len=16, window=8, hi_budget=7)
    compare(s, np.array(cu, np.int32), pol)
    compare(s[:3000], np.array([0, 1200, 3000], np.int32), pol)


def test_many_one_token_sequences():
    T = 300
    s = np.random.default_rng(3).random(T).astype(np.float32)
    pol = wl.Policy.ladder([8, 16, 32, 64], 32.0, [0.25, 0.5, 0.75], min_len=1, window=0, max_len=1)
    ref = compare(s, np.arange(T + 1, dtype=np.int32), pol)
    assert ref.n_chunks == T and np.all(ref.flags == 1)


def test_empty_input_and_capacity_overflow():
    pol = wl.Policy.ladder([4, 8], 8.0, [0.5], min_len=4, window=0)
    got, status = run(np.zeros(0, np.float32), np.array([0, 0], np.int32), pol)
    assert status == 0 and got["n_chunks"] == 0 and got["offsets"].tolist() == [0]
    s = np.random.default_rng(1).random(400).astype(np.float32)
    got, status = run(s, np.array([0, 400], np.int32), wl.Policy.ladder([4, 8], 8.0, [0.5], 4, 0, max_len=4), capacity=10)
    assert status == (1 << 4) and got["n_chunks"] == 0        # CWL_ERR_CAPACITY raised, table marked empty


def test_bad_policy_is_rejected():
    st = torch.zeros(8, dtype=torch.float32, device="cuda")
    cu = torch.tensor([0, 8], dtype=torch.int32, device="cuda")
    bad = cwl.make_policy([8, 4], [1, 1], [0.5], 2, 4, 0)       # ranks must not decrease
    with pytest.raises(cwl.CwlError):
        cwl.cwl_partition(st, cu, bad)
