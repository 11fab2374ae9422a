"""Pins of the oracle's chunker and selector (Sec. III-B, III-C).

The paper prints neither a decision rule nor a worked example for the chunker, so parity with
the paper is unpinned; what is pinned here: the fixed-point rung against exact rational
arithmetic, hand-traced partitions, the invariants the length bounds and the budget imply, and an
independent brute-force restatement (first-stop search over exact fractions, no prefix sums)."""
from fractions import Fraction

import numpy as np
import pytest

import oracle

Q = 1 << 24
LADDER3 = dict(ranks=[4, 8, 16], scales=[4.0, 2.0, 1.0], thresholds=[0.33, 0.66])


# ------------------------------------------------------------------ independent brute force
def bf_quant(s):
    s = np.float32(s)
    if np.isnan(s):
        return Q
    f = Fraction(float(min(max(s, np.float32(0)), np.float32(1))))
    return (f * Q).__floor__()


def bf_rung(qs, thresholds):
    """Rung of a span from exact rationals: number of thresholds its mean reaches."""
    mean = Fraction(sum(qs), len(qs))
    return sum(1 for th in thresholds if mean >= (Fraction(float(np.float32(th))) * Q).__floor__())


def bf_partition(score, cu, ranks, scales, thresholds, min_len, max_len, hi_budget=-1):
    q = [bf_quant(s) for s in score]
    offsets, rungs, flags = [0], [], []
    for n in range(len(cu) - 1):
        S, E = int(cu[n]), int(cu[n + 1])
        seq_chunks = []
        b = S
        while b < E:
            cut = E
            if E - b >= 2 * min_len:
                # candidates keep a legal tail; the first one that must close the chunk wins
                for e in range(b + min_len, E - min_len + 1):
                    capped = (e - b) >= max_len
                    changes = bf_rung(q[b:e], thresholds) != bf_rung(q[e:e + min_len], thresholds)
                    if capped or changes:
                        cut = e
                        break
            seq_chunks.append((b, cut))
            b = cut
        rs = [bf_rung(q[b:e], thresholds) for b, e in seq_chunks]
        K = len(ranks)
        if hi_budget >= 0 and K >= 2:
            top = [i for i, r in enumerate(rs) if r == K - 1]
            # largest mean first, earlier chunk first on ties
            order = sorted(top, key=lambda i: (-Fraction(sum(q[seq_chunks[i][0]:seq_chunks[i][1]]),
                                                         seq_chunks[i][1] - seq_chunks[i][0]), i))
            for i in order[hi_budget:]:
                rs[i] = K - 2
        for i, (b, e) in enumerate(seq_chunks):
            offsets.append(e)
            rungs.append(rs[i])
            flags.append(1 if i == 0 else 0)
    return offsets, rungs, flags


def check_equal(tab, bf, ranks, scales):
    offsets, rungs, flags = bf
    assert tab.offsets.tolist() == offsets
    assert tab.rung.tolist() == rungs
    assert tab.flags.tolist() == flags
    assert tab.rank.tolist() == [ranks[r] for r in rungs]
    assert tab.scale.tolist() == [np.float32(scales[r]) for r in rungs]


# ------------------------------------------------------------------ quantise and rung
def test_quantise_values():
    assert oracle.quantise(0.0) == 0
    assert oracle.quantise(1.0) == Q
    assert oracle.quantise(2.5) == Q
    assert oracle.quantise(-0.1) == 0
    assert oracle.quantise(float("nan")) == Q
    assert oracle.quantise(0.5) == Q // 2
    assert oracle.quantise(np.float32(2.0 ** -24)) == 1
    assert oracle.quantise(np.float32(2.0 ** -25)) == 0
    rng = np.random.default_rng(0)
    for s in rng.random(200).astype(np.float32):
        assert oracle.quantise(s) == bf_quant(s)


def test_rung_exhaustive_small():
    ths = [0.25, 0.5, 0.75]
    ranks, scales = [1, 2, 3, 4], [1, 1, 1, 1]
    for length in range(1, 5):
        for k in range(0, 4 * length + 1):
            for delta in (-1, 0, 1):
                total = k * (Q // 4) * 1 + delta
                if total < 0 or total > Q * length:
                    continue
                want = sum(1 for th in ths if Fraction(total, length) >= int(th * Q))
                assert oracle.rung_of(total, length, ranks, scales, ths) == want


def test_rung_single_token_is_threshold_compare_and_monotone():
    ths = LADDER3["thresholds"]
    rng = np.random.default_rng(1)
    s = np.sort(rng.random(500).astype(np.float32))
    r = [oracle.rung_of(oracle.quantise(v), 1, LADDER3["ranks"], LADDER3["scales"], ths) for v in s]
    assert r == sorted(r)
    for v, k in zip(s, r):
        # away from a threshold's quantisation cell the fixed-point compare is the plain compare
        if all(abs(float(v) - float(np.float32(t))) > 2.0 / Q for t in ths):
            assert k == sum(1 for t in ths if v >= np.float32(t))


# ------------------------------------------------------------------ hand-traced partitions
def test_constant_score_gives_max_len_chunks_then_tail_rule():
    T, Lmin, Lmax = 100, 4, 16
    s = np.full(T, 0.5, np.float32)
    tab = oracle.partition(s, [0, T], **LADDER3, min_len=Lmin, max_len=Lmax)
    # 16,16,16,16,16,16 then 4 left: 96..100; at b=80: E-b=20, candidates up to e=96 -> cut at 96 (cap);
    # at b=96: E-b=4 < 2*Lmin -> takes the rest
    assert tab.offsets.tolist() == [0, 16, 32, 48, 64, 80, 96, 100]
    assert set(tab.rung.tolist()) == {1}
    T = 99  # at b=80: E-b=19, candidates e in 84..95 none stops (len<16, same rung) -> absorbs to 99
    tab = oracle.partition(np.full(T, 0.5, np.float32), [0, T], **LADDER3, min_len=Lmin, max_len=Lmax)
    assert tab.offsets.tolist() == [0, 16, 32, 48, 64, 80, 99]


def test_clean_step_cuts_at_the_step():
    Lmin, Lmax = 8, 128
    for p in (8, 13, 40):
        s = np.concatenate([np.full(p, 0.1), np.full(64, 0.9)]).astype(np.float32)
        tab = oracle.partition(s, [0, len(s)], **LADDER3, min_len=Lmin, max_len=Lmax)
        # look-ahead window [e, e+8) reaches rung 1 when it holds 4 of 8 hard tokens, i.e. e = p - 4 ... but the
        # open chunk must have len >= 8; the cut is the first e >= 8 whose window class differs from rung 0.
        mean_ok = [e for e in range(Lmin, len(s) - Lmin + 1)
                   if bf_rung([bf_quant(v) for v in s[:e]], LADDER3["thresholds"]) !=
                   bf_rung([bf_quant(v) for v in s[e:e + Lmin]], LADDER3["thresholds"])]
        assert tab.offsets[1] == mean_ok[0]
        # window mean (k*0.9 + (8-k)*0.1) >= 0.33 first at k = 3 hard tokens -> e = p - 5 (when >= Lmin)
        assert tab.offsets[1] == max(Lmin, p - 5)
    # a step that is already in place when the chunk may first close (p <= L_min): cut at L_min
    s = np.concatenate([np.full(8, 0.1), np.full(64, 0.9)]).astype(np.float32)
    assert oracle.partition(s, [0, 72], **LADDER3, min_len=8, max_len=128).offsets[1] == 8


def test_short_sequences_are_one_chunk():
    for L in (1, 7, 8, 15):
        rng = np.random.default_rng(L)
        s = rng.random(L).astype(np.float32)
        tab = oracle.partition(s, [0, L], **LADDER3, min_len=8, max_len=128)
        assert tab.offsets.tolist() == [0, L] and tab.flags.tolist() == [1]
    tab = oracle.partition(np.zeros(0, np.float32), [0, 0], **LADDER3, min_len=8, max_len=128)
    assert tab.n_chunks == 0 and tab.offsets.tolist() == [0]
    # empty sequences between non-empty ones emit nothing
    s = np.full(10, 0.2, np.float32)
    tab = oracle.partition(s, [0, 0, 4, 4, 10, 10], **LADDER3, min_len=8, max_len=128)
    assert tab.offsets.tolist() == [0, 4, 10] and tab.flags.tolist() == [1, 1]


# ------------------------------------------------------------------ invariants, brute force
def random_case(rng, max_T=64):
    n_seq = int(rng.integers(1, 4))
    lens = rng.integers(0, max_T // n_seq + 1, size=n_seq)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(cu[-1])
    kind = rng.integers(0, 3)
    if kind == 0:
        s = rng.random(T)
    elif kind == 1:  # piecewise constant + noise
        s = np.repeat(rng.random(T // 5 + 1), 5)[:T] + rng.normal(0, 0.03, T)
    else:            # coarse grid: many exact ties at the thresholds
        s = rng.integers(0, 5, T) / 4.0
    s = s.astype(np.float32)
    if T and rng.random() < 0.2:
        s[rng.integers(0, T)] = np.nan
    K = int(rng.integers(1, 5))
    ranks = sorted(rng.choice([0, 2, 4, 8, 16, 32], size=K, replace=False).tolist())
    scales = [float(np.float32(16.0 / r)) if r else 0.0 for r in ranks]
    ths = sorted(rng.choice([0.1, 0.25, 0.33, 0.5, 0.66, 0.75, 0.9], size=K - 1, replace=False).tolist())
    min_len = int(rng.integers(1, 6))
    max_len = min_len + int(rng.integers(0, 12))
    hi_budget = int(rng.choice([-1, 0, 1, 2, 3]))
    return s, cu, dict(ranks=ranks, scales=scales, thresholds=ths, min_len=min_len, max_len=max_len,
                       hi_budget=hi_budget)


@pytest.mark.parametrize("seed", range(60))
def test_matches_brute_force_and_invariants(seed):
    rng = np.random.default_rng(1000 + seed)
    s, cu, kw = random_case(rng)
    tab = oracle.partition(s, cu, **kw)
    bf = bf_partition(s, cu, kw["ranks"], kw["scales"], kw["thresholds"], kw["min_len"], kw["max_len"],
                      kw["hi_budget"])
    check_equal(tab, bf, kw["ranks"], kw["scales"])
    # invariants of the length bounds (Sec. III-B)
    off = tab.offsets
    T = int(cu[-1])
    assert off[0] == 0 and off[-1] == T and np.all(np.diff(off) > 0)
    bounds = set(int(c) for c in cu)
    seq_of = np.searchsorted(cu, off[:-1], side="right") - 1
    for c in range(tab.n_chunks):
        b, e = int(off[c]), int(off[c + 1])
        n = int(seq_of[c])
        S, E = int(cu[n]), int(cu[n + 1])
        assert S <= b and e <= E                        # never crosses a sequence boundary
        assert (tab.flags[c] & 1) == (1 if b == S else 0)
        if E - S >= kw["min_len"]:
            assert e - b >= kw["min_len"]
        if e < E:
            assert e - b <= kw["max_len"]
        else:
            assert e - b < kw["max_len"] + kw["min_len"]
    assert bounds.issuperset({0, T})
    # budget: at most H top-rung chunks per sequence
    K = len(kw["ranks"])
    if kw["hi_budget"] >= 0 and K >= 2:
        for n in range(len(cu) - 1):
            assert int(np.sum((seq_of == n) & (tab.rung == K - 1))) <= kw["hi_budget"]


def test_packed_batch_is_concatenation_of_single_sequences():
    rng = np.random.default_rng(7)
    lens = [37, 0, 64, 5, 120]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    s = (np.repeat(rng.random(60), 4)[:cu[-1]] + rng.normal(0, 0.02, cu[-1])).clip(0, 0.999).astype(np.float32)
    kw = dict(**LADDER3, min_len=4, max_len=32, hi_budget=2)
    packed = oracle.partition(s, cu, **kw)
    offs, rungs, flags = [0], [], []
    for n, L in enumerate(lens):
        one = oracle.partition(s[cu[n]:cu[n + 1]], [0, L], **kw)
        offs += (one.offsets[1:] + cu[n]).tolist()
        rungs += one.rung.tolist()
        flags += one.flags.tolist()
    assert packed.offsets.tolist() == offs and packed.rung.tolist() == rungs and packed.flags.tolist() == flags


def test_budget_demotes_lowest_means_first():
    # five well separated hard spans with means 0.95, 0.80, 0.90, 0.70, 0.85 between easy stretches
    means = [0.95, 0.80, 0.90, 0.70, 0.85]
    parts = []
    for m in means:
        parts += [np.full(16, 0.1), np.full(16, m)]
    s = np.concatenate(parts).astype(np.float32)
    base = oracle.partition(s, [0, len(s)], **LADDER3, min_len=4, max_len=16, hi_budget=-1)
    top = np.nonzero(base.rung == 2)[0]
    assert len(top) >= 5
    for H in (0, 1, 3, 99):
        tab = oracle.partition(s, [0, len(s)], **LADDER3, min_len=4, max_len=16, hi_budget=H)
        assert tab.offsets.tolist() == base.offsets.tolist()          # the budget never re-cuts
        keep = np.nonzero(tab.rung == 2)[0]
        assert len(keep) == min(H, len(top))
        sums = np.array([s[base.offsets[c]:base.offsets[c + 1]].astype(np.float64).mean() for c in top])
        kept_means = sorted(sums[np.isin(top, keep)])
        assert kept_means == sorted(sums)[len(top) - len(keep):]
        demoted = np.setdiff1d(top, keep)
        assert np.all(tab.rung[demoted] == 1)


def test_budget_tie_goes_to_earlier_chunk():
    s = np.concatenate([np.full(8, 0.1), np.full(8, 0.9), np.full(8, 0.1), np.full(8, 0.9)]).astype(np.float32)
    tab = oracle.partition(s, [0, 32], **LADDER3, min_len=8, max_len=8, hi_budget=1)
    assert tab.offsets.tolist() == [0, 8, 16, 24, 32]
    assert tab.rung.tolist() == [0, 2, 0, 1]


def test_bad_arguments_are_rejected():
    s = np.zeros(8, np.float32)
    with pytest.raises(ValueError):
        oracle.partition(s, [0, 8], **LADDER3, min_len=0, max_len=4)
    with pytest.raises(ValueError):
        oracle.partition(s, [0, 8], **LADDER3, min_len=4, max_len=2)
    with pytest.raises(ValueError):
        oracle.partition(s, [0, 8], **LADDER3, min_len=4, max_len=8, window=5)
    with pytest.raises(ValueError):
        oracle.partition(s, [0, 5, 3, 8], **LADDER3, min_len=4, max_len=8)
    with pytest.raises(ValueError):
        oracle.partition(s, [0, 8], ranks=[4, 8], scales=[1, 1], thresholds=[0.7, 0.2][:1] + [], min_len=4,
                         max_len=8, window=9)
    with pytest.raises(OverflowError):
        oracle.partition(s, [0, 8], **LADDER3, min_len=1, max_len=1, capacity=3)
