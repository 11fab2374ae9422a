"""Pins of the oracle's centred cross-fade window (Sec. III-D variant: the window lies around the join, the last
floor(w/2) rows of the outgoing chunk and the first ceil(w/2) rows of the incoming one): a hand-expanded tiny
case, the ramp's closed form, its relation to the causal placement, and the structural properties a blend must
have (convex combination of single-configuration runs, invisible between equal neighbours)."""
import os

import numpy as np
import pytest

import oracle
from paper_2601_21109_b200.workloads import f32_to_bf16_bits
from test_oracle_apply import GOLDEN, f64, problem, table


def test_hand_expanded_tiny_case():
    vals = {}
    with open(os.path.join(GOLDEN, "apply_centred_tiny.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, *nums = line.split()
            vals[key] = np.array([float(v) for v in nums])
    X = f32_to_bf16_bits(vals["X"].reshape(5, 2).astype(np.float32))
    W = f32_to_bf16_bits(vals["W"].reshape(2, 2).astype(np.float32))
    A = f32_to_bf16_bits(vals["A"].reshape(2, 2).astype(np.float32))
    B = f32_to_bf16_bits(vals["B"].reshape(2, 2).astype(np.float32))
    tab = table(vals["offsets"].astype(int), vals["rank"].astype(int), vals["scale"], vals["flags"].astype(int))
    Y = oracle.apply(X, W, A, B, tab, int(vals["window"][0]), centred=True)
    assert Y.reshape(-1).tolist() == vals["Y"].tolist()


@pytest.mark.parametrize("w", [0, 1, 2, 3, 4, 5, 8])
def test_ramp_closed_form_and_window_sums(w):
    # chunks of 8..12 rows, two sequences: joins at 10, 18 (sequence 0) and 40 (sequence 1); 30 starts sequence 1
    tab = table([0, 10, 18, 30, 40, 52], [4, 8, 2, 8, 4], [1, 1, 1, 1, 1], flags=[1, 0, 0, 1, 0])
    lam, cin, cout = oracle.blend_weights_centred(tab, 52, w)
    before, after = w // 2, w - w // 2
    expected_rows = set()
    for join, c in ((10, 1), (18, 2), (40, 4)):
        rows = list(range(join - before, join + after))
        expected_rows.update(rows)
        assert lam[rows].tolist() == [(i + 1) / (w + 1) for i in range(w)]      # equally spaced, strictly inside (0,1)
        assert abs(lam[rows].sum() - w / 2) < 1e-12                             # the two ramps share the window equally
        assert all(cin[r] == c and cout[r] == c - 1 for r in rows)              # both sides blend (c-1 out, c in)
    others = [t for t in range(52) if t not in expected_rows]
    assert np.all(lam[others] == 1.0) and np.all(cin[others] == cout[others])
    # no window across the sequence boundary at row 30
    assert lam[29] == 1.0 and lam[30] == 1.0


@pytest.mark.parametrize("w", [1, 2, 4, 5])
def test_same_ramp_as_the_causal_placement_shifted_back(w):
    tab = table([0, 12, 24], [4, 8], [1, 1])
    causal = oracle.blend_weights(tab, 24, w)
    centred, _, _ = oracle.blend_weights_centred(tab, 24, w)
    shift = w // 2
    assert centred[12 - shift:12 - shift + w].tolist() == causal[12:12 + w].tolist()


def test_short_chunk_gives_its_rows_to_the_opening_join():
    # chunk 1 has 3 rows, window 4: after = 2 rows of the window that opens it, before = 2 rows of the one that closes it;
    # row 1 of the chunk is claimed by both: the opening join's window wins, the closing join keeps the last row only
    tab = table([0, 6, 9, 15], [4, 8, 2], [1, 1, 1])
    lam, cin, cout = oracle.blend_weights_centred(tab, 15, 4)
    assert (cin[6], cout[6], lam[6]) == (1, 0, 3 / 5) and (cin[7], cout[7], lam[7]) == (1, 0, 4 / 5)
    assert (cin[8], cout[8], lam[8]) == (2, 1, 2 / 5)
    assert (cin[9], cout[9], lam[9]) == (2, 1, 3 / 5) and (cin[10], cout[10], lam[10]) == (2, 1, 4 / 5)


def test_window_rows_are_convex_combinations_of_single_configuration_runs():
    X, W, A, B = problem(11, T=30)
    w = 5
    tab = table([0, 9, 21, 30], [8, 2, 5], [0.5, 3.0, 1.25])
    Y = oracle.apply(X, W, A, B, tab, w, centred=True)
    lam, cin, cout = oracle.blend_weights_centred(tab, 30, w)
    single = [oracle.apply(X, W, A, B, table([0, 30], [int(tab.rank[c])], [float(tab.scale[c])]), 0) for c in range(3)]
    for t in range(30):
        want = (1.0 - lam[t]) * single[cout[t]][t] + lam[t] * single[cin[t]][t]
        np.testing.assert_allclose(Y[t], want, rtol=1e-12, atol=1e-12)
    assert sum(1 for t in range(30) if lam[t] < 1.0) == 2 * w


def test_zero_window_and_equal_neighbours_show_no_window():
    X, W, A, B = problem(12, T=24)
    tab = table([0, 8, 16, 24], [4, 4, 8], [1.5, 1.5, 0.5])
    np.testing.assert_array_equal(oracle.apply(X, W, A, B, tab, 0, centred=True), oracle.apply(X, W, A, B, tab, 0))
    Yc = oracle.apply(X, W, A, B, tab, 4, centred=True)
    Y0 = oracle.apply(X, W, A, B, tab, 0)
    np.testing.assert_allclose(Yc[:14], Y0[:14], rtol=1e-12, atol=1e-12)     # the join at 8 joins equal configurations
    assert np.abs(Yc[14:18] - Y0[14:18]).max() > 1e-3                         # the join at 16 does not


def test_row_subset_mode_and_dense_mode():
    X, W, A, B = problem(13, T=20)
    tab = table([0, 10, 20], [8, 3], [1.0, 2.0])
    full = oracle.apply(X, W, A, B, tab, 4, centred=True)
    rows = np.array([19, 8, 9, 10, 11, 0], np.int32)
    np.testing.assert_array_equal(oracle.apply(X, W, A, B, tab, 4, rows=rows, centred=True), full[rows])
    np.testing.assert_allclose(oracle.apply(X, W, None, None, None, 0, centred=True), f64(X) @ f64(W), rtol=1e-13, atol=1e-13)
