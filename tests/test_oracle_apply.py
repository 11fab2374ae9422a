"""Pins of the oracle's cross-fade (Sec. III-D) and adapted projection (Sec. III-F) against the
textbook merged-weight LoRA, the frozen base, a hand-expanded tiny case and structural
properties (linearity, prefix slicing, convex combination of single-configuration runs)."""
import os

import numpy as np
import pytest

import oracle
from oracle import ChunkTable
from paper_2601_21109_b200.workloads import bf16_bits_to_f32, f32_to_bf16_bits, normal_bf16

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f64(bits):
    return bf16_bits_to_f32(bits).astype(np.float64)


def table(offsets, rank, scale, flags=None):
    n = len(rank)
    fl = np.array(flags if flags is not None else [1] + [0] * (n - 1), np.int32)
    return ChunkTable(np.array(offsets, np.int32), np.array(rank, np.int32), np.array(scale, np.float32),
                      np.zeros(n, np.int32), fl, n)


def problem(seed, T=23, d_in=12, d_out=9, R=8):
    rng = np.random.default_rng(seed)
    return (normal_bf16(rng, (T, d_in), 1.0), normal_bf16(rng, (d_in, d_out), 0.3),
            normal_bf16(rng, (d_in, R), 0.3), normal_bf16(rng, (R, d_out), 0.4))


def test_bf16_helpers_round_to_nearest_even():
    x = np.array([1.0, 1.00390625, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -2.5, 0.0], np.float32)
    back = bf16_bits_to_f32(f32_to_bf16_bits(x))
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: even mantissa (1.0) wins; 1 + 3*2^-8 ties up to 1 + 2^-6
    assert back.tolist() == [1.0, 1.0, 1.0, 1.0 + 2 ** -6, -2.5, 0.0]


def test_hand_expanded_tiny_case():
    vals = {}
    with open(os.path.join(GOLDEN, "apply_tiny.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, *nums = line.split()
            vals[key] = np.array([float(v) for v in nums])
    X = f32_to_bf16_bits(vals["X"].reshape(3, 2).astype(np.float32))
    W = f32_to_bf16_bits(vals["W"].reshape(2, 2).astype(np.float32))
    A = f32_to_bf16_bits(vals["A"].reshape(2, 2).astype(np.float32))
    B = f32_to_bf16_bits(vals["B"].reshape(2, 2).astype(np.float32))
    tab = table(vals["offsets"].astype(int), vals["rank"].astype(int), vals["scale"], vals["flags"].astype(int))
    Y = oracle.apply(X, W, A, B, tab, int(vals["window"][0]))
    assert Y.reshape(-1).tolist() == vals["Y"].tolist()


def test_full_rank_equals_merged_weight_lora():
    X, W, A, B = problem(0)
    T, R = X.shape[0], A.shape[1]
    alpha = 16.0
    Y = oracle.apply(X, W, A, B, table([0, T], [R], [alpha / R]), window=4)
    merged = f64(W) + (alpha / R) * (f64(A) @ f64(B))
    np.testing.assert_allclose(Y, f64(X) @ merged, rtol=1e-12, atol=1e-12)


def test_rank_zero_and_no_adapter_equal_base():
    X, W, A, B = problem(1)
    T = X.shape[0]
    base = f64(X) @ f64(W)
    np.testing.assert_allclose(oracle.apply(X, W, A, B, table([0, T], [0], [3.0]), 2), base, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(oracle.apply(X, W, None, None, None, 0), base, rtol=1e-13, atol=1e-13)


def test_prefix_slicing_of_the_ladder():
    X, W, A, B = problem(2)
    T = X.shape[0]
    for r in (1, 3, 8):
        Y = oracle.apply(X, W, A, B, table([0, T], [r], [0.75]), 0)
        want = f64(X) @ f64(W) + 0.75 * (f64(X) @ f64(A)[:, :r]) @ f64(B)[:r, :]
        np.testing.assert_allclose(Y, want, rtol=1e-12, atol=1e-12)


def test_single_chunk_has_no_boundary_effect():
    X, W, A, B = problem(3)
    T = X.shape[0]
    tab = table([0, T], [4], [2.0])
    y0 = oracle.apply(X, W, A, B, tab, 0)
    for w in (1, 4, 16):
        assert np.array_equal(oracle.apply(X, W, A, B, tab, w), y0)


def test_blend_weights_are_a_linear_ramp_that_sums_to_one():
    T = 40
    tab = table([0, 10, 18, 30, 40], [2, 4, 8, 2], [1, 1, 1, 1], flags=[1, 0, 1, 0])
    for w in (0, 1, 4, 8):
        lam = oracle.blend_weights(tab, T, w)
        assert np.all((lam > 0) & (lam <= 1))
        out_w = 1.0 - lam                                   # weight of the outgoing configuration
        np.testing.assert_allclose(out_w + lam, 1.0, atol=0)
        for c, blended in ((1, True), (2, False), (3, True)):
            o = tab.offsets[c]
            win = lam[o:o + w]
            if blended and w:
                np.testing.assert_allclose(win.sum(), w / 2.0, rtol=1e-15)          # symmetric ramp
                np.testing.assert_allclose(np.diff(np.concatenate([[0.0], win, [1.0]])), 1.0 / (w + 1), rtol=1e-12)
            else:
                assert np.all(win == 1.0)
        mask = np.ones(T, bool)
        for c in (1, 3):
            mask[tab.offsets[c]:tab.offsets[c] + w] = False
        assert np.all(lam[mask] == 1.0)


def test_window_rows_are_convex_combinations_of_single_configuration_runs():
    X, W, A, B = problem(4, T=30)
    T = X.shape[0]
    tab = table([0, 12, 30], [8, 2], [0.5, 4.0])
    w = 5
    Y = oracle.apply(X, W, A, B, tab, w)
    y_out = oracle.apply(X, W, A, B, table([0, T], [8], [0.5]), 0)      # outgoing configuration everywhere
    y_in = oracle.apply(X, W, A, B, table([0, T], [2], [4.0]), 0)       # incoming configuration everywhere
    np.testing.assert_allclose(Y[:12], y_out[:12], rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(Y[12 + w:], y_in[12 + w:], rtol=1e-13, atol=1e-13)
    for j in range(w):
        lam = (j + 1) / (w + 1)
        np.testing.assert_allclose(Y[12 + j], (1 - lam) * y_out[12 + j] + lam * y_in[12 + j], rtol=1e-12, atol=1e-12)
    # w = 0: piecewise, no blending at all
    Y0 = oracle.apply(X, W, A, B, tab, 0)
    np.testing.assert_allclose(Y0[12:], y_in[12:], rtol=1e-13, atol=1e-13)


def test_equal_neighbours_hide_the_window_and_sequence_starts_do_not_blend():
    X, W, A, B = problem(5, T=30)
    same = table([0, 12, 30], [4, 4], [2.0, 2.0])
    one = table([0, 30], [4], [2.0])
    np.testing.assert_allclose(oracle.apply(X, W, A, B, same, 6), oracle.apply(X, W, A, B, one, 6), rtol=1e-13, atol=1e-13)
    first = table([0, 12, 30], [8, 2], [0.5, 4.0], flags=[1, 1])        # second chunk starts a new sequence
    y_in = oracle.apply(X, W, A, B, table([0, 30], [2], [4.0]), 0)
    np.testing.assert_allclose(oracle.apply(X, W, A, B, first, 6)[12:], y_in[12:], rtol=1e-13, atol=1e-13)


def test_gate_form_equals_literal_blend_and_scale_is_linear():
    X, W, A, B = problem(6, T=26, R=8)
    tab = table([0, 7, 15, 26], [2, 8, 4], [4.0, 1.0, 2.0])
    w = 3
    Y = oracle.apply(X, W, A, B, tab, w)
    # gate form: y = xW + ((xA) * g) B with g[j] = (1-lam) s_p [j<r_p] + lam s_c [j<r_c]
    lam = oracle.blend_weights(tab, 26, w)
    H = f64(X) @ f64(A)
    G = np.zeros_like(H)
    for t in range(26):
        c = int(np.searchsorted(tab.offsets, t, side="right") - 1)
        j = np.arange(8)
        G[t] = lam[t] * tab.scale[c] * (j < tab.rank[c])
        if lam[t] < 1:
            G[t] += (1 - lam[t]) * tab.scale[c - 1] * (j < tab.rank[c - 1])
    np.testing.assert_allclose(Y, f64(X) @ f64(W) + (H * G) @ f64(B), rtol=1e-12, atol=1e-12)
    # doubling every scale doubles the adapter part
    base = f64(X) @ f64(W)
    tab2 = table([0, 7, 15, 26], [2, 8, 4], [8.0, 2.0, 4.0])
    np.testing.assert_allclose(oracle.apply(X, W, A, B, tab2, w) - base, 2 * (Y - base), rtol=1e-11, atol=1e-11)


def test_row_subset_mode_matches_full_run():
    X, W, A, B = problem(7, T=33)
    tab = table([0, 9, 20, 33], [8, 2, 4], [1.0, 4.0, 2.0])
    Y = oracle.apply(X, W, A, B, tab, 4)
    rows = np.array([32, 0, 9, 10, 12, 13, 20, 21, 5], np.int32)
    assert np.array_equal(oracle.apply(X, W, A, B, tab, 4, rows=rows), Y[rows])


def test_bad_tables_are_rejected():
    X, W, A, B = problem(8)
    T = X.shape[0]
    with pytest.raises(ValueError):
        oracle.apply(X, W, A, B, table([0, T - 1], [4], [1.0]), 0)          # does not cover T
    with pytest.raises(ValueError):
        oracle.apply(X, W, A, B, table([0, T], [9], [1.0]), 0)              # rank above R
    with pytest.raises(ValueError):
        oracle.apply(X, W, A, B, table([0, T], [4], [1.0]), 0, rows=np.array([T], np.int32))
