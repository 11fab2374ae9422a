"""Pins of the oracle's mixed complexity score (Sec. III-A: entropy, n-gram novelty against the recent
context, positional prior).  The paper lists the signals without formulas; the definitions are pinned by
special cases that reduce to known quantities, a hand-traced token stream and a set-based brute force."""
import numpy as np
import pytest

import oracle


def flat_logits(T, V=16):
    return np.zeros((T, V), dtype=np.float32)          # entropy score exactly 1 on every row


def novelty(ids, cu, n, ctx):
    ids = np.asarray(ids, np.int32)
    return oracle.score_tokens_mixed(flat_logits(len(ids)), ids, np.asarray(cu, np.int32), 0.0, 1.0, 0.0, n, ctx, 1)


def test_entropy_only_is_the_plain_score():
    rng = np.random.default_rng(0)
    z = (rng.standard_normal((40, 50)) * 2.5).astype(np.float32)
    ids = rng.integers(0, 9, 40)
    got = oracle.score_tokens_mixed(z, ids, [0, 40], 1.0, 0.0, 0.0, 2, 8, 10)
    assert np.array_equal(got, oracle.score_tokens(z))


def test_hand_traced_bigram_novelty():
    ids = [1, 2, 3, 1, 2, 3, 1, 2, 4]
    # bigrams ending at t: -, (1,2), (2,3), (3,1), (1,2)*, (2,3)*, (3,1)*, (1,2)*, (2,4); * = seen before
    assert novelty(ids, [0, 9], 2, 8).tolist() == [1, 1, 1, 1, 0, 0, 0, 0, 1]
    # a context of two positions no longer reaches the earlier occurrence three tokens back
    assert novelty(ids, [0, 9], 2, 2).tolist() == [1] * 9
    # the context of exactly three positions does
    assert novelty(ids, [0, 9], 2, 3).tolist() == [1, 1, 1, 1, 0, 0, 0, 0, 1]


def test_unigram_novelty_and_sequence_boundaries():
    ids = [5, 6, 5, 7, 5, 6, 5, 7]
    assert novelty(ids, [0, 8], 1, 8).tolist() == [1, 1, 0, 1, 0, 0, 0, 0]
    # the same stream as two sequences of four tokens: nothing is matched across the boundary
    assert novelty(ids, [0, 4, 8], 1, 8).tolist() == [1, 1, 0, 1, 1, 1, 0, 1]
    # bigrams never reach across the boundary either: (7|5) is not a bigram of the second sequence
    assert novelty([1, 2, 1, 2, 1, 2], [0, 3, 6], 2, 8).tolist() == [1, 1, 1, 1, 1, 1]


def test_positional_prior_closed_form():
    T = 12
    got = oracle.score_tokens_mixed(flat_logits(T), np.zeros(T, np.int32), [0, 7, 12], 0.0, 0.0, 1.0, 1, 4, 5)
    want = [max(0.0, 1 - p / 5) for p in range(7)] + [max(0.0, 1 - p / 5) for p in range(5)]
    assert np.allclose(got, want, rtol=0, atol=1e-15)


def test_mix_is_the_clamped_weighted_sum():
    rng = np.random.default_rng(1)
    T = 60
    z = (rng.standard_normal((T, 30)) * 3).astype(np.float32)
    ids = rng.integers(0, 4, T)
    cu = [0, 25, 60]
    e = oracle.score_tokens_mixed(z, ids, cu, 1.0, 0.0, 0.0, 2, 16, 20)
    n = oracle.score_tokens_mixed(z, ids, cu, 0.0, 1.0, 0.0, 2, 16, 20)
    p = oracle.score_tokens_mixed(z, ids, cu, 0.0, 0.0, 1.0, 2, 16, 20)
    w = (np.float32(0.5), np.float32(0.3), np.float32(0.2))
    got = oracle.score_tokens_mixed(z, ids, cu, *map(float, w), 2, 16, 20)
    assert np.allclose(got, np.clip(float(w[0]) * e + float(w[1]) * n + float(w[2]) * p, 0, 1), rtol=0, atol=1e-15)
    big = oracle.score_tokens_mixed(z, ids, cu, 1.0, 1.0, 1.0, 2, 16, 20)
    assert big.max() == 1.0 and big.min() >= 0.0                       # clamped


@pytest.mark.parametrize("seed", range(6))
def test_novelty_matches_set_based_brute_force(seed):
    rng = np.random.default_rng(50 + seed)
    n, ctx = int(rng.integers(1, 5)), int(rng.integers(1, 40))
    lens = rng.integers(1, 60, size=5)
    cu = np.concatenate([[0], np.cumsum(lens)])
    ids = rng.integers(0, 3, cu[-1])                                   # tiny alphabet: many repeats
    want = []
    for s in range(5):
        seq = ids[cu[s]:cu[s + 1]].tolist()
        for p in range(len(seq)):
            if p < n - 1:
                want.append(1.0)
                continue
            gram = tuple(seq[p - n + 1:p + 1])
            earlier = {tuple(seq[u - n + 1:u + 1]) for u in range(max(n - 1, p - ctx), p)}
            want.append(0.0 if gram in earlier else 1.0)
    assert novelty(ids, cu, n, ctx).tolist() == want


def test_nan_entropy_stays_nan_and_bad_arguments():
    z = flat_logits(3)
    z[1, 2] = np.nan
    got = oracle.score_tokens_mixed(z, [1, 2, 3], [0, 3], 0.5, 0.25, 0.25, 1, 2, 2)
    assert np.isnan(got[1]) and not np.isnan(got[[0, 2]]).any()
    with pytest.raises(ValueError):
        oracle.score_tokens_mixed(z, [1, 2, 3], [0, 3], 0.5, 0.25, 0.25, 0, 2, 2)
    with pytest.raises(ValueError):
        oracle.score_tokens_mixed(z, [1, 2, 3], [0, 2], 0.5, 0.25, 0.25, 1, 2, 2)
