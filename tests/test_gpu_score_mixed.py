"""GPU parity of cwl_score_tokens_mixed (Sec. III-A: entropy + n-gram novelty + positional prior) against the
oracle, through the C ABI: fp32 scores within 1e-5 relative (floor 1e-2), the novelty bit itself exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run(z, ids, cu, *mix):
    s = cwl.cwl_score_tokens_mixed(torch.from_numpy(z).cuda(), torch.from_numpy(np.asarray(ids, np.int32)).cuda(),
                                   torch.from_numpy(np.asarray(cu, np.int32)).cuda(), *mix)
    return s.cpu().numpy().astype(np.float64)


def close(got, ref):
    both_nan = np.isnan(got) & np.isnan(ref)
    err = np.abs(got - ref) / np.maximum(np.abs(ref), 1e-2)
    assert np.all(both_nan | (err <= 1e-5)), float(np.nanmax(err))


@pytest.mark.parametrize("seed", range(5))
def test_random_streams_all_signals(seed):
    rng = np.random.default_rng(900 + seed)
    lens = rng.integers(1, 400, size=int(rng.integers(1, 7)))
    cu = np.concatenate([[0], np.cumsum(lens)])
    T, V = int(cu[-1]), int(rng.choice([64, 1000, 4099]))
    z = wl.span_temperature_logits(rng, T, V)
    ids = rng.integers(0, int(rng.choice([3, 50])), T)
    n, ctx, span = int(rng.integers(1, 5)), int(rng.choice([1, 7, 300, 1000])), int(rng.choice([1, 64, 5000]))
    w = rng.dirichlet([1, 1, 1]).astype(np.float32)
    mix = (float(w[0]), float(w[1]), float(w[2]), n, ctx, span)
    close(run(z, ids, cu, *mix), oracle.score_tokens_mixed(z, ids, cu, *mix))
    # the novelty bit on its own is an exact integer decision
    nov = run(np.zeros((T, 8), np.float32), ids, cu, 0.0, 1.0, 0.0, n, ctx, span)
    assert np.array_equal(nov, oracle.score_tokens_mixed(np.zeros((T, 8), np.float32), ids, cu, 0.0, 1.0, 0.0, n, ctx, span))


def test_entropy_weight_one_reproduces_cwl_score_tokens_bits():
    rng = np.random.default_rng(3)
    z = wl.span_temperature_logits(rng, 300, 32000)
    zt = torch.from_numpy(z).cuda()
    ids = torch.zeros(300, dtype=torch.int32, device="cuda")
    cu = torch.tensor([0, 300], dtype=torch.int32, device="cuda")
    a = cwl.cwl_score_tokens(zt)
    b = cwl.cwl_score_tokens_mixed(zt, ids, cu, 1.0, 0.0, 0.0, 2, 16, 100)
    assert torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_config2_size_with_a_long_context():
    rng = np.random.default_rng(wl.SEED_BASE + 2)
    T, V = 2048, 32000
    z = wl.span_temperature_logits(rng, T, V)
    ids = rng.integers(0, 200, T)
    mix = (0.6, 0.3, 0.1, 3, 512, 2048)
    got = run(z, ids, [0, T], *mix)
    rows = np.unique(np.concatenate([[0, 1, 2, T - 1], rng.integers(0, T, 96)]))
    # the novelty of a row depends on its whole context, so the oracle scores the full stream (seconds at this size)
    full = oracle.score_tokens_mixed(z, ids, [0, T], *mix)
    close(got[rows], full[rows])
    close(got, full)


def test_nan_row_and_bad_arguments():
    z = np.zeros((4, 16), np.float32)
    z[2, 3] = np.inf
    got = run(z, [1, 1, 1, 1], [0, 4], 0.5, 0.25, 0.25, 1, 4, 4)
    assert np.isnan(got[2]) and not np.isnan(got[[0, 1, 3]]).any()
    zt = torch.from_numpy(z).cuda()
    ids = torch.zeros(4, dtype=torch.int32, device="cuda")
    cu = torch.tensor([0, 4], dtype=torch.int32, device="cuda")
    for bad in [(0.5, 0.5, 0.0, 0, 4, 4), (0.5, -0.1, 0.0, 1, 4, 4), (0.5, 0.5, 0.0, 1, 0, 4), (0.5, 0.5, 0.0, 9, 4, 4)]:
        with pytest.raises(cwl.CwlError):
            cwl.cwl_score_tokens_mixed(zt, ids, cu, *bad)
