"""GPU parity of cwl_batch_align (Sec. III-G, IV-F: sequences bucketed by complexity percentile share their chunk
joins) against the oracle, bit for bit, through the C ABI: buckets, order, offsets, rungs, ranks, scales, flags."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def compare(score, cu, pol: wl.Policy, n_buckets, capacity=None):
    st = torch.from_numpy(np.ascontiguousarray(score, np.float32)).cuda()
    cut = torch.from_numpy(np.ascontiguousarray(cu, np.int32)).cuda()
    cp = cwl.make_policy(pol.ranks, pol.scales, pol.thresholds, pol.min_len, pol.max_len, pol.window, pol.hi_budget)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    table = None if capacity is None else cwl.DeviceChunkTable(capacity)
    tab, bucket, pos = cwl.cwl_batch_align(st, cut, cp, n_buckets, table=table, status_word=status)
    torch.cuda.synchronize()
    got = tab.to_host()
    if capacity is not None:
        return got, int(status.item())
    assert int(status.item()) == 0
    ref, rb, rp = oracle.batch_align(score, cu, pol.ranks, pol.scales, pol.thresholds, pol.min_len, pol.max_len, n_buckets,
                                     pol.window, pol.hi_budget)
    assert np.array_equal(bucket.cpu().numpy(), rb) and np.array_equal(pos.cpu().numpy(), rp)
    assert got["n_chunks"] == ref.n_chunks
    for key in ("offsets", "rank", "rung"):
        assert np.array_equal(got[key], getattr(ref, key)), key
    assert np.array_equal(got["flags"] & 1, ref.flags & 1)
    assert np.array_equal(got["scale"].view(np.uint32), ref.scale.view(np.uint32))
    return ref


@pytest.mark.parametrize("seed", range(24))
def test_random_batches_and_policies(seed):
    rng = np.random.default_rng(8100 + seed)
    n_seq = int(rng.integers(1, 40))
    lens = rng.integers(0, 500, size=n_seq)
    if seed % 4 == 0:
        lens[rng.integers(0, n_seq)] = 0
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(cu[-1])
    level = np.repeat(rng.uniform(0, 1, n_seq), lens)
    s = np.clip(level + 0.3 * np.sin(np.arange(T) / rng.uniform(3, 40)) + rng.normal(0, 0.05, T), -0.1, 1.1).astype(np.float32)
    if T and seed % 5 == 0:
        s[rng.integers(0, T)] = np.nan
    min_len = int(rng.integers(1, 33))
    pol = wl.Policy.ladder([4, 8, 16, 32], 16.0, sorted(rng.uniform(0.1, 0.9, 3).tolist()), min_len=min_len,
                           window=0, max_len=min_len * int(rng.integers(1, 9)), hi_budget=int(rng.choice([-1, 0, 1, 3])))
    compare(s, cu, pol, int(rng.choice([1, 2, 3, 8, n_seq, n_seq + 5])))


def test_config3_packed_batch_in_four_buckets():
    w = wl.config3(d=16)
    ref = compare(w.score, w.cu_seqlens, w.policy, 4)
    assert ref.n_chunks > 200
    # one bucket per sequence: the table of cwl_partition
    p = w.policy
    alone = compare(w.score, w.cu_seqlens, w.policy, len(w.cu_seqlens) - 1)
    part = oracle.partition(w.score, w.cu_seqlens, p.ranks, p.scales, p.thresholds, p.min_len, p.max_len, p.window, p.hi_budget)
    assert np.array_equal(alone.offsets, part.offsets) and np.array_equal(alone.rank, part.rank)


def test_long_sequences_one_bucket():
    rng = np.random.default_rng(5)
    lens = [9000, 20000, 3, 15000]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(cu[-1])
    s = np.clip(np.repeat(rng.uniform(0, 1, T // 50 + 1), 50)[:T] + rng.normal(0, 0.05, T), 0, 1).astype(np.float32)
    compare(s, cu, wl.Policy.ladder([8, 16, 32, 64], 32.0, [0.25, 0.5, 0.75], min_len=16, window=8), 1)


def test_capacity_overflow_and_bad_arguments():
    s = np.linspace(0, 1, 64).astype(np.float32)
    pol = wl.Policy.ladder([4, 8], 8.0, [0.5], min_len=2, window=0, max_len=2)
    got, status = compare(s, [0, 64], pol, 1, capacity=3)
    assert got["n_chunks"] == 0 and status == 1 << 4
    st = torch.from_numpy(s).cuda()
    cu = torch.tensor([0, 64], dtype=torch.int32, device="cuda")
    cp = cwl.make_policy(pol.ranks, pol.scales, pol.thresholds, 2, 2, 0, -1)
    with pytest.raises(cwl.CwlError) as e:
        cwl.cwl_batch_align(st, cu, cp, 0)
    assert e.value.status == 1
    with pytest.raises(cwl.CwlError) as e:
        cwl.cwl_batch_align(st, cu, cp, 4096)
    assert e.value.status == 3
    # no sequences at all
    tab, b, p = cwl.cwl_batch_align(torch.empty(0, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda"), cp, 2)
    torch.cuda.synchronize()
    assert tab.to_host()["n_chunks"] == 0
