"""Pins of the oracle's offline ladder construction (Sec. III-C: prefix slices of SVD-ordered factors).
The SVD itself is a library routine; what is pinned is that the factors it is turned into have the
properties the method relies on, each checked by an independent computation."""
import numpy as np

import oracle
from paper_2601_21109_b200 import workloads as wl


def factors(seed, d_in=48, d_out=40, R=8, decay=None):
    rng = np.random.default_rng(seed)
    A = rng.standard_normal((d_in, R)).astype(np.float32)
    if decay is not None:
        A *= decay ** np.arange(R, dtype=np.float32)
    B = rng.standard_normal((R, d_out)).astype(np.float32) * 0.3
    return wl.f32_to_bf16_bits(A), wl.f32_to_bf16_bits(B)


def f64(bits):
    return wl.bf16_bits_to_f32(bits).astype(np.float64)


def test_product_is_preserved_and_prefixes_are_best_approximations():
    A, B = factors(1, decay=0.6)
    dW = f64(A) @ f64(B)
    A2, B2, s = oracle.svd_ladder(A, B)
    assert np.allclose(A2 @ B2, dW, rtol=0, atol=1e-12 * np.abs(dW).max())
    assert np.all(np.diff(s) <= 0) and s[-1] >= 0
    assert np.allclose(B2 @ B2.T, np.eye(B2.shape[0]), atol=1e-12)                 # right factors orthonormal
    assert np.allclose(np.linalg.norm(A2, axis=0), s, rtol=1e-12)                  # left factors carry sigma
    for r in range(0, len(s)):
        err = dW - A2[:, :r] @ B2[:r, :]
        # Eckart-Young: the error of the best rank-r approximation is sigma_{r+1} in the 2-norm ...
        assert np.isclose(np.linalg.norm(err, 2), s[r], rtol=1e-9)
        # ... and the root of the remaining squared singular values in the Frobenius norm
        assert np.isclose(np.linalg.norm(err, "fro"), np.sqrt(np.sum(s[r:] ** 2)), rtol=1e-9)


def test_no_rank_r_product_of_the_original_slices_beats_the_ladder():
    # prefix slices of the UNORDERED trained factors are worse (or equal) than the ladder's at every rank
    A, B = factors(2)
    dW = f64(A) @ f64(B)
    A2, B2, _ = oracle.svd_ladder(A, B)
    for r in range(1, A2.shape[1]):
        naive = np.linalg.norm(dW - f64(A)[:, :r] @ f64(B)[:r, :], "fro")
        ladder = np.linalg.norm(dW - A2[:, :r] @ B2[:r, :], "fro")
        assert ladder <= naive * (1 + 1e-12)


def test_diagonal_case_closed_form():
    # A = columns of the identity scaled by (1, 2, 4, 8), B = rows of the identity: sigma = (8, 4, 2, 1)
    A = np.zeros((6, 4), np.float32); B = np.zeros((4, 5), np.float32)
    for j, v in enumerate([1.0, 2.0, 4.0, 8.0]):
        A[j, j] = v; B[j, j] = 1.0
    A2, B2, s = oracle.svd_ladder(wl.f32_to_bf16_bits(A), wl.f32_to_bf16_bits(B))
    assert np.allclose(s, [8, 4, 2, 1])
    assert np.allclose(np.abs(A2[:4, :4]), np.diag([1.0, 2.0, 4.0, 8.0])[:, ::-1])
    assert np.allclose(A2 @ B2, A.astype(np.float64) @ B.astype(np.float64))


def test_rank_deficient_update():
    A, B = factors(3, R=6)
    A[:, 5] = A[:, 0]                      # a repeated direction: the update has rank 5
    B[5, :] = B[1, :]
    A2, B2, s = oracle.svd_ladder(A, B)
    dW = f64(A) @ f64(B)
    assert s[5] <= 1e-10 * s[0]
    assert np.allclose(A2[:, :5] @ B2[:5, :], dW, atol=1e-10 * np.abs(dW).max())
