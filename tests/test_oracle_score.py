"""Pins of the oracle's token score (next-token entropy, Sec. III-A signal (i)) against closed
forms, invariances and a library routine -- none of them the oracle's own formula re-typed."""
import math

import numpy as np
import pytest

import oracle


def test_constant_row_is_maximal_entropy():
    for V in (2, 7, 1000, 32000):
        for c in (0.0, -3.5, 11.0):
            z = np.full((1, V), c, np.float32)
            assert oracle.score_tokens(z)[0] == 1.0


@pytest.mark.parametrize("V,k,a", [(10, 1, 2.0), (100, 3, 5.0), (32000, 2, 9.0), (17, 16, 1.5)])
def test_k_equal_maxima_closed_form(V, k, a):
    # k logits at a over a zero floor: p_max = e^a / Z each, p_rest = 1 / Z each, Z = k e^a + V - k
    z = np.zeros((1, V), np.float32)
    z[0, :k] = a
    Z = k * math.exp(a) + (V - k)
    H = math.log(Z) - k * a * math.exp(a) / Z
    got = oracle.score_tokens(z)[0]
    # 32000 sequential fp64 additions: allow V * 2^-53 of drift
    assert got == pytest.approx(H / math.log(V), rel=1e-11, abs=1e-15)


def test_peaked_limits():
    V = 50
    z = np.zeros((2, V), np.float32)
    z[0, 3] = 80.0                      # one-hot limit: entropy -> 0
    z[1, 3] = 80.0
    z[1, 9] = 80.0                      # two equal peaks: entropy -> ln 2
    s = oracle.score_tokens(z)
    assert s[0] == pytest.approx(0.0, abs=1e-30)
    assert s[1] == pytest.approx(math.log(2.0) / math.log(V), rel=1e-13)


def test_shift_and_permutation_invariance():
    rng = np.random.default_rng(1)
    z = (rng.standard_normal((4, 257)) * 2.0).astype(np.float32)
    # snap to a 2^-10 grid below 8 in magnitude so that z + 16 is exact in fp32
    z = np.clip(np.round(z * 1024) / 1024, -7.5, 7.5).astype(np.float32)
    s = oracle.score_tokens(z)
    shifted = (z + np.float32(16.0)).astype(np.float32)
    assert np.array_equal(shifted.astype(np.float64), z.astype(np.float64) + 16.0)
    np.testing.assert_allclose(oracle.score_tokens(shifted), s, rtol=1e-13)
    perm = rng.permutation(z.shape[1])
    np.testing.assert_allclose(oracle.score_tokens(z[:, perm]), s, rtol=1e-12)


def test_two_way_reduces_to_binary_entropy():
    d = np.array([-6.0, -1.25, 0.0, 0.5, 3.0, 10.0])
    z = np.stack([np.zeros_like(d), d], axis=1).astype(np.float32)
    p = 1.0 / (1.0 + np.exp(-d))
    Hb = -(p * np.log(p) + (1 - p) * np.log1p(-p))
    np.testing.assert_allclose(oracle.score_tokens(z), Hb / math.log(2.0), rtol=1e-12, atol=1e-15)


def test_gaussian_logits_small_sigma_expansion():
    # For z ~ N(0, sigma^2) and large V: H ~ ln V - sigma^2 / 2 (second-order cumulant expansion)
    rng = np.random.default_rng(2)
    V = 32000
    for sigma in (0.25, 0.5, 1.0):
        z = (rng.standard_normal((16, V)) * sigma).astype(np.float32)
        s = oracle.score_tokens(z)
        assert abs(s.mean() - (1.0 - sigma * sigma / (2.0 * math.log(V)))) < 1e-3


def test_against_library_log_softmax():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(3)
    z = (rng.standard_normal((8, 1234)) / rng.uniform(0.3, 3.0, size=(8, 1))).astype(np.float32)
    lp = torch.log_softmax(torch.from_numpy(z).double(), dim=-1)
    H = -(lp.exp() * lp).sum(-1).numpy()
    np.testing.assert_allclose(oracle.score_tokens(z), H / math.log(z.shape[1]), rtol=1e-12)


def test_special_values():
    V = 8
    z = np.zeros((5, V), np.float32)
    z[0, 2] = -np.inf                     # zero-probability entry: entropy of the other V-1
    z[1, 0] = np.nan
    z[2, 5] = np.inf
    z[3, :] = -np.inf
    z[4, 1:] = -np.inf                    # a single finite entry: entropy 0
    s = oracle.score_tokens(z)
    assert s[0] == pytest.approx(math.log(V - 1) / math.log(V), rel=1e-14)
    assert np.isnan(s[1]) and np.isnan(s[2]) and np.isnan(s[3])
    assert s[4] == 0.0


def test_range_and_order():
    # flatter rows (higher temperature) score higher
    rng = np.random.default_rng(4)
    g = rng.standard_normal((1, 4000)).astype(np.float32)
    taus = [0.3, 0.6, 1.0, 2.0, 3.0]
    s = [oracle.score_tokens((g / t).astype(np.float32))[0] for t in taus]
    assert all(0.0 <= v <= 1.0 for v in s)
    assert all(a < b for a, b in zip(s, s[1:]))
