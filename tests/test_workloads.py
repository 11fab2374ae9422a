"""The seeded generators: deterministic, right shapes and structure, and the oracle runs on them."""
import numpy as np

import oracle
from paper_2601_21109_b200 import workloads as wl


def test_config1_is_deterministic_and_has_planted_spans():
    a, b = wl.config1(), wl.config1()
    assert np.array_equal(a.score, b.score) and np.array_equal(a.projections[0].W, b.projections[0].W)
    assert a.T == 256 and a.X[1024].shape == (256, 1024) and a.projections[0].B.shape == (16, 1024)
    for s in a.notes["planted_starts"]:
        assert np.all(a.score[s:s + 24] >= 0.8)
    assert a.score.max() < 1.0 and a.score.min() >= 0.0
    p = a.policy
    assert p.ranks == [4, 8, 16] and p.scales == [4.0, 2.0, 1.0] and p.min_len == 8 and p.window == 4
    tab = oracle.partition(a.score, a.cu_seqlens, p.ranks, p.scales, p.thresholds, p.min_len, p.max_len, p.window)
    # every planted span sits (mostly) on the top rung
    for s in a.notes["planted_starts"]:
        c = np.searchsorted(tab.offsets, s + 12, side="right") - 1
        assert tab.rank[c] == 16


def test_config2_small_variant_scores_in_expected_band():
    w = wl.config2(T=256, V=2000, projections=[("q", 64, 64)])
    assert w.logits.shape == (256, 2000) and w.logits.dtype == np.float32
    s = oracle.score_tokens(w.logits)
    assert 0.3 < s.min() and s.max() <= 1.0
    # one temperature per 64-token span: scores are nearly constant inside a span
    assert np.all(s.reshape(4, 64).std(axis=1) < 0.02)


def test_config3_lengths_and_regimes():
    w = wl.config3(d=32)
    lens = np.diff(w.cu_seqlens)
    assert len(lens) == 32 and lens.min() >= 128 and lens.max() <= 4096 and w.T == int(lens.sum())
    assert 20000 < w.T < 60000
    assert w.score.shape == (w.T,) and 0.0 <= w.score.min() and w.score.max() < 1.0
    p = w.policy
    tab = oracle.partition(w.score, w.cu_seqlens, p.ranks, p.scales, p.thresholds, p.min_len, p.max_len, p.window)
    assert tab.n_chunks <= w.T // p.min_len + 32
    assert len(set(tab.rank.tolist())) >= 4          # the regimes exercise most of the ladder


def test_config4_table_is_one_chunk_per_row():
    w = wl.config4(T=16)
    t = w.table
    assert t["offsets"].tolist() == list(range(17)) and np.all(t["flags"] == 1)
    assert set(t["rank"].tolist()) <= {8, 16, 32, 64}
    np.testing.assert_array_equal(t["scale"], np.float32(32.0) / t["rank"].astype(np.float32))


def test_static_table_and_row_sampling():
    t = wl.static_table(np.array([0, 5, 5, 9]), 64, 32.0)
    assert t["offsets"].tolist() == [0, 5, 9] and t["rank"].tolist() == [64, 64] and t["scale"].tolist() == [0.5, 0.5]
    rng = np.random.default_rng(0)
    rows = wl.sample_rows(rng, 100, np.array([0, 20, 50, 100]), np.array([1, 0, 0]), window=4)
    assert rows[0] == 0 and rows[-1] == 99 and np.all(np.diff(rows) > 0)
    assert {20, 21, 22, 23}.issubset(set(rows.tolist())) or {50, 51, 52, 53}.issubset(set(rows.tolist()))
