"""Pins of the oracle's batch alignment (Sec. III-G, IV-F: sequences bucketed by complexity percentile share
their chunk joins).  The paper gives one sentence and no rule, so parity with it is unpinned; pinned here: the
reduction to the (pinned) per-sequence chunker when every sequence is its own bucket or when the members of a
bucket are identical, a pooled walk traced by hand, the properties the reading implies (a permutation, buckets
monotone in mean and of near-equal size, joins shared inside a bucket, length bounds, per-sequence rungs) and an
independent brute force over exact fractions written from the text."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from test_oracle_partition import bf_quant, bf_rung

POL = dict(ranks=[4, 8, 16], scales=[4.0, 2.0, 1.0], thresholds=[0.25, 0.75])


def align(score, cu, n_buckets, min_len=4, max_len=12, hi_budget=-1, pol=POL):
    return oracle.batch_align(np.asarray(score, np.float32), np.asarray(cu, np.int32), pol["ranks"], pol["scales"],
                              pol["thresholds"], min_len, max_len, n_buckets, 0, hi_budget)


def part(score, cu, min_len=4, max_len=12, hi_budget=-1, pol=POL):
    return oracle.partition(np.asarray(score, np.float32), np.asarray(cu, np.int32), pol["ranks"], pol["scales"],
                            pol["thresholds"], min_len, max_len, 0, hi_budget)


def tables_equal(a, b):
    return (a.n_chunks == b.n_chunks and np.array_equal(a.offsets, b.offsets) and np.array_equal(a.rank, b.rank)
            and np.array_equal(a.rung, b.rung) and np.array_equal(a.flags & 1, b.flags & 1)
            and np.array_equal(a.scale, b.scale))


def random_batch(rng, n_seq, max_seq_len=90):
    lens = rng.integers(0, max_seq_len, size=n_seq)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    level = np.repeat(rng.uniform(0, 1, size=n_seq), lens)
    wave = 0.3 * np.sin(np.arange(cu[-1]) / rng.uniform(3, 9))
    s = np.clip(level + wave + rng.normal(0, 0.05, cu[-1]), 0, 1).astype(np.float32)
    return s, cu


@pytest.mark.parametrize("seed", range(12))
def test_one_bucket_per_sequence_is_the_per_sequence_chunker(seed):
    rng = np.random.default_rng(100 + seed)
    n_seq = int(rng.integers(1, 9))
    s, cu = random_batch(rng, n_seq)
    budget = int(rng.choice([-1, 0, 1, 2]))
    tab, bucket, pos = align(s, cu, n_seq, hi_budget=budget)
    assert tables_equal(tab, part(s, cu, hi_budget=budget))
    assert sorted(bucket.tolist()) == list(range(n_seq)) and np.array_equal(bucket, pos)


def test_identical_members_of_a_bucket_keep_their_own_partition():
    rng = np.random.default_rng(7)
    one = np.clip(rng.uniform(0, 1, 57) + np.repeat(rng.uniform(-0.4, 0.4, 19), 3), 0, 1).astype(np.float32)
    s = np.tile(one, 3)
    cu = np.array([0, 57, 114, 171], np.int32)
    tab, bucket, pos = align(s, cu, 1, hi_budget=1)
    assert tables_equal(tab, part(s, cu, hi_budget=1))
    assert bucket.tolist() == [0, 0, 0] and pos.tolist() == [0, 1, 2]          # ties keep the index order


def test_hand_traced_pooled_walk():
    # Two sequences in ONE bucket, eighths: L = 1/8, H = 7/8.  L_min = 4, L_max = 12, thresholds 0.25 / 0.75.
    #   seq 0 (16 tokens): L L L L  L L L L  H H H H  H H H H
    #   seq 1 (12 tokens): H H H H  L L L L  L L L L
    # pooled track, positions 0..15: N = 2 for j < 12, 1 after.  S (in eighths): j<4: 8, 4..7: 2, 8..11: 8, 12..15: 7
    #   b=0: e=4: pooled mean [0,4) = 32/8 / 8 = 1/2 -> rung 1; ahead [4,8): 8/8 / 8 = 1/8 -> rung 0: cut at 4
    #   b=4: e=8: [4,8) rung 0; ahead [8,12): 1/2 -> rung 1: cut at 8
    #   b=8: 8 tokens left (= 2 L_min): e=12: [8,12) mean 1/2 -> rung 1; ahead [12,16): 28/8 / 4 = 7/8 -> rung 2: cut at 12
    #   b=12: 4 left (< 2 L_min): rest.  Shared joins: 4, 8, 12.
    # seq 0 (len 16) takes 4, 8, 12 (12 <= 16 - 4); seq 1 (len 12) takes 4 and 8 (8 <= 12 - 4; 12 is its end).
    # Own rungs: seq 0: L->0, L->0, H->2, H->2;  seq 1: H->2, L->0, L->0.
    L, H = 0.125, 0.875
    s = [L] * 8 + [H] * 8 + [H] * 4 + [L] * 8
    tab, bucket, pos = align(s, [0, 16, 28], 1)
    assert tab.offsets.tolist() == [0, 4, 8, 12, 16, 20, 24, 28]
    assert tab.rung.tolist() == [0, 0, 2, 2, 2, 0, 0]
    assert tab.rank.tolist() == [4, 4, 16, 16, 16, 4, 4]
    assert (tab.flags & 1).tolist() == [1, 0, 0, 0, 1, 0, 0]
    # on its own, sequence 0 is cut where ITS look-ahead window first leaves rung 0 (position 5: L L L H has mean
    # 10/32 >= 1/4); aligned, it follows the bucket's joins instead
    assert part(s[:16], [0, 16]).offsets.tolist()[:2] == [0, 5]
    # mean of seq 0 = 1/2, of seq 1 = (4*7 + 8*1)/96 = 3/8: seq 1 comes first in the complexity order
    assert pos.tolist() == [1, 0] and bucket.tolist() == [0, 0]


def test_percentile_buckets_are_monotone_and_balanced():
    rng = np.random.default_rng(3)
    s, cu = random_batch(rng, 23)
    for nb in (1, 2, 4, 5, 23):
        tab, bucket, pos = align(s, cu, nb)
        assert sorted(pos.tolist()) == list(range(23))                        # a permutation
        assert np.array_equal(bucket, pos * nb // 23)
        sizes = np.bincount(bucket, minlength=nb)
        assert sizes.max() - sizes.min() <= 1
        # bucket index never decreases along the complexity order, and the order is by exact mean
        q = np.array([bf_quant(x) for x in s], dtype=object)
        means = [Fraction(int(q[cu[n]:cu[n + 1]].sum()), int(cu[n + 1] - cu[n])) if cu[n + 1] > cu[n] else Fraction(-1)
                 for n in range(23)]
        by_pos = np.argsort(pos)
        assert all(means[by_pos[i]] <= means[by_pos[i + 1]] for i in range(22))
        assert all(bucket[by_pos[i]] <= bucket[by_pos[i + 1]] for i in range(22))


def bf_align(score, cu, thresholds, min_len, max_len, n_buckets):
    """Joins per sequence from the text of the reading: exact fractions, no prefix sums."""
    q = [bf_quant(x) for x in score]
    n_seq = len(cu) - 1
    lens = [int(cu[n + 1] - cu[n]) for n in range(n_seq)]
    key = [(0, Fraction(0), n) if lens[n] == 0 else (1, Fraction(sum(q[cu[n]:cu[n + 1]]), lens[n]), n) for n in range(n_seq)]
    order = sorted(range(n_seq), key=lambda n: key[n])
    bucket = [0] * n_seq
    for i, n in enumerate(order):
        bucket[n] = i * n_buckets // n_seq
    cuts_of = {}
    for k in set(bucket):
        members = [n for n in range(n_seq) if bucket[n] == k]
        Lk = max(lens[n] for n in members)
        pooled = [[q[cu[n] + j] for n in members if lens[n] > j] for j in range(Lk)]

        def rung(b, e):
            vals = [v for col in pooled[b:e] for v in col]
            return bf_rung(vals, thresholds)
        joins, b = [], 0
        while b < Lk:
            cut = Lk
            if Lk - b >= 2 * min_len:
                for e in range(b + min_len, Lk - min_len + 1):
                    if (e - b) >= max_len or rung(b, e) != rung(e, e + min_len):
                        cut = e
                        break
            if cut < Lk:
                joins.append(cut)
            b = cut
        cuts_of[k] = joins
    offsets = [0]
    for n in range(n_seq):
        if lens[n] == 0:
            continue
        offsets += [int(cu[n]) + c for c in cuts_of[bucket[n]] if c <= lens[n] - min_len] + [int(cu[n + 1])]
    return offsets, bucket


@pytest.mark.parametrize("seed", range(30))
def test_against_a_brute_force_over_exact_fractions(seed):
    rng = np.random.default_rng(900 + seed)
    n_seq = int(rng.integers(1, 10))
    s, cu = random_batch(rng, n_seq, max_seq_len=70)
    nb = int(rng.integers(1, n_seq + 1))
    min_len = int(rng.integers(1, 7))
    max_len = min_len * int(rng.integers(1, 5))
    tab, bucket, _ = align(s, cu, nb, min_len=min_len, max_len=max_len)
    want_offsets, want_bucket = bf_align(s, cu, POL["thresholds"], min_len, max_len, nb)
    assert bucket.tolist() == want_bucket
    assert tab.offsets.tolist() == want_offsets
    # rung of every chunk from the sequence's own scores
    q = [bf_quant(x) for x in s]
    for c in range(tab.n_chunks):
        assert tab.rung[c] == bf_rung(q[tab.offsets[c]:tab.offsets[c + 1]], POL["thresholds"])


@pytest.mark.parametrize("seed", range(8))
def test_members_share_joins_and_keep_the_length_bounds(seed):
    rng = np.random.default_rng(40 + seed)
    n_seq = 12
    s, cu = random_batch(rng, n_seq, max_seq_len=120)
    min_len, max_len = 5, 20
    tab, bucket, _ = align(s, cu, 3, min_len=min_len, max_len=max_len)
    first = np.flatnonzero(tab.flags & 1)
    assert tab.offsets[first].tolist() == [int(cu[n]) for n in range(n_seq) if cu[n + 1] > cu[n]]   # chunks never cross sequences
    joins = {}
    for n in range(n_seq):
        lo, hi = int(cu[n]), int(cu[n + 1])
        inner = [int(o) - lo for o in tab.offsets if lo < o < hi]
        joins[n] = inner
        lens = np.diff([0] + inner + [hi - lo]) if hi > lo else []
        for i, l in enumerate(lens):
            assert l >= min_len or len(lens) == 1
            assert l <= max_len or (i == len(lens) - 1 and l < max_len + min_len)
    for k in range(3):
        members = [n for n in range(n_seq) if bucket[n] == k and cu[n + 1] > cu[n]]
        longest = max(members, key=lambda n: cu[n + 1] - cu[n])
        for n in members:
            limit = int(cu[n + 1] - cu[n]) - min_len
            assert joins[n] == [j for j in joins[longest] if j <= limit]      # the bucket's joins, cut off by the length


def test_bad_arguments():
    with pytest.raises(ValueError):
        align([0.5] * 8, [0, 8], 0)
    with pytest.raises(ValueError):
        align([0.5] * 8, [0, 9], 1)
    tab, bucket, pos = align([], [0], 3)
    assert tab.n_chunks == 0
