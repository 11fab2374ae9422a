"""GPU parity of cwl_score_tokens (entropy signal, Sec. III-A (i)) against the fp64 oracle:
fp32 scores within 1e-5 relative (floored at |s| = 1e-2, where a relative bound on a value
that tends to 0 stops being meaningful)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_scores
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def check(z: np.ndarray, ld=None):
    zt = torch.from_numpy(z).cuda()
    if ld is not None:
        buf = torch.zeros(z.shape[0], ld, dtype=torch.float32, device="cuda")
        buf[:, :z.shape[1]] = zt
        zt = buf[:, :z.shape[1]]
    s = cwl.cwl_score_tokens(zt).cpu().numpy().astype(np.float64)
    ref = oracle.score_tokens(z)
    return check_scores(s, ref, label=f"score {z.shape[0]}x{z.shape[1]}")


def test_temperature_spans_llama_vocab():
    rng = np.random.default_rng(1)
    check(wl.span_temperature_logits(rng, 192, 32000))


@pytest.mark.parametrize("V", [2, 3, 5, 127, 1000, 4099, 32003])
def test_odd_vocab_sizes_and_unaligned_rows(V):
    rng = np.random.default_rng(V)
    z = (rng.standard_normal((37, V)) * rng.uniform(0.3, 4.0, size=(37, 1))).astype(np.float32)
    check(z)                 # rows start at arbitrary 4-byte offsets when V is odd
    check(z, ld=V + 5)


def test_special_values_and_peaked_rows():
    V = 513
    rng = np.random.default_rng(9)
    z = rng.standard_normal((10, V)).astype(np.float32)
    z[0, 5] = -np.inf
    z[1, 7] = np.nan
    z[2, 9] = np.inf
    z[3, :] = -np.inf
    z[4, 1:] = -np.inf
    z[5, :] = 3.25                       # constant row: exactly 1
    z[6, 100] = 60.0                     # near one-hot
    z[7, :256] = -np.inf                 # leading -inf block, then finite
    z[8, :] *= 30.0                      # very peaked
    z[9, :] = -1e30
    check(z)
    s = cwl.cwl_score_tokens(torch.from_numpy(z).cuda()).cpu().numpy()
    assert s[5] == pytest.approx(1.0, abs=2e-6) and s[4] == 0.0


def test_config2_full_size_sampled_rows():
    rng = np.random.default_rng(wl.SEED_BASE + 2)
    z = wl.span_temperature_logits(rng, 2048, 32000)
    zt = torch.from_numpy(z).cuda()
    s = cwl.cwl_score_tokens(zt).cpu().numpy().astype(np.float64)
    rows = np.unique(np.concatenate([[0, 2047], np.random.default_rng(0).integers(0, 2048, 128)]))
    ref = oracle.score_tokens(z[rows])
    check_scores(s[rows], ref, label="score cfg2 full size, sampled rows")
    assert np.all((s >= 0.3) & (s <= 1.0))


def test_empty_and_bad_arguments():
    z = torch.zeros(0, 16, dtype=torch.float32, device="cuda")
    assert cwl.cwl_score_tokens(z).shape == (0,)
    with pytest.raises(cwl.CwlError):
        cwl.cwl_score_tokens(torch.zeros(4, 1, dtype=torch.float32, device="cuda"))   # V < 2
