"""GPU parity of cwl_ladder_build (Sec. III-C: SVD-ordered adapter factors) against the oracle.  Singular vectors
are unique only up to sign, so what is compared is what is unique: the singular values and every prefix product
A'[:, :r] B'[:r, :] of the ladder's ranks; the factors' own properties (orthonormal rows of B', column norms of A')
are checked directly."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import dev_bf16
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def trained_factors(rng, d_in, d_out, R, decay):
    A = rng.standard_normal((d_in, R)).astype(np.float32) * d_in ** -0.5 * decay ** np.arange(R, dtype=np.float32)
    B = rng.standard_normal((R, d_out)).astype(np.float32) * R ** -0.5
    return wl.f32_to_bf16_bits(A), wl.f32_to_bf16_bits(B)


def check(A, B, ranks):
    out = cwl.cwl_ladder_build(dev_bf16(A), dev_bf16(B))
    torch.cuda.synchronize()
    A_ref, B_ref, s_ref = oracle.svd_ladder(A, B)
    s = out["sigma"].cpu().numpy().astype(np.float64)
    A2, B2 = out["A32"].cpu().numpy().astype(np.float64), out["B32"].cpu().numpy().astype(np.float64)
    scale = s_ref[0]
    assert np.all(np.diff(s) <= 0)
    assert np.max(np.abs(s - s_ref)) <= 1e-5 * scale
    assert np.max(np.abs(B2 @ B2.T - np.eye(len(s)))[s_ref > 1e-6 * scale][:, s_ref > 1e-6 * scale]) <= 1e-5
    assert np.max(np.abs(np.linalg.norm(A2, axis=0) - s_ref)) <= 1e-5 * scale
    dW = A_ref @ B_ref
    for r in ranks:
        got, ref = A2[:, :r] @ B2[:r, :], A_ref[:, :r] @ B_ref[:r, :]
        assert np.linalg.norm(got - ref) <= 1e-5 * np.linalg.norm(dW), r
    # the bf16 copies are the fp32 results rounded once
    a16 = wl.bf16_bits_to_f32(out["A"].view(torch.int16).cpu().numpy().view(np.uint16))
    assert np.array_equal(a16, wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(out["A32"].cpu().numpy())))
    return out


def test_small_ladder():
    rng = np.random.default_rng(1)
    A, B = trained_factors(rng, 96, 80, 16, 0.8)
    out = check(A, B, [4, 8, 16])
    assert 1 <= out["sweeps"] <= 60


def test_llama_sized_projection_R64():
    rng = np.random.default_rng(2)
    A, B = trained_factors(rng, 4096, 11008, 64, 0.93)
    check(A, B, [8, 16, 32, 64])


def test_rank_deficient_update():
    rng = np.random.default_rng(3)
    A, B = trained_factors(rng, 128, 96, 16, 1.0)
    A[:, 15] = A[:, 0]
    B[15, :] = B[3, :]
    out = check(A, B, [4, 8, 15, 16])
    assert float(out["sigma"][15]) <= 1e-5 * float(out["sigma"][0])


def test_ladder_feeds_the_adapted_projection():
    # prefix slices of the rebuilt factors through cwl_apply: rank R reproduces the trained adapter's output
    from gpu_util import check_output, dev_table, y_to_f64
    rng = np.random.default_rng(4)
    T, d_in, d_out, R = 160, 256, 192, 16
    A, B = trained_factors(rng, d_in, d_out, R, 0.7)
    X = wl.normal_bf16(rng, (T, d_in), 1.0)
    W = wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5)
    out = cwl.cwl_ladder_build(dev_bf16(A), dev_bf16(B))
    tab = dict(offsets=np.array([0, T], np.int32), rank=np.array([R], np.int32), scale=np.array([1.0], np.float32),
               flags=np.array([1], np.int32), rung=np.zeros(1, np.int32), n_chunks=1)
    Y = cwl.cwl_apply(dev_bf16(X), dev_bf16(W), out["A"], out["B"], dev_table(tab), 0)
    ref = oracle.apply(X, W, A, B, oracle.ChunkTable(tab["offsets"], tab["rank"], tab["scale"], tab["rung"], tab["flags"], 1), 0)
    check_output(y_to_f64(Y), ref)


def test_argument_errors():
    A = torch.zeros(64, 15, dtype=torch.bfloat16, device="cuda")
    B = torch.zeros(15, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(cwl.CwlError) as e:
        cwl.cwl_ladder_build(A, B)                      # odd R
    assert e.value.status == 3
