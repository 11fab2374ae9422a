"""cwl_apply_noalloc: the variant of the adapted projection for callers that cannot allocate device
memory (its scratch is a fixed array inside the library).  Collected last on purpose.

Checked through the C ABI against the ordinary cwl_apply on the same inputs, on two calls in a row
with different shapes and tables, so that whatever the first call leaves in the shared scratch must
not leak into the second."""
import gc

import numpy as np
import pytest
import torch

from gpu_util import check_output, dev_bf16, dev_table, y_to_f64
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def case(seed, T, d_in, d_out, R, cuts, ranks, scales, window):
    rng = np.random.default_rng(seed)
    X = dev_bf16(wl.normal_bf16(rng, (T, d_in), 1.0))
    W = dev_bf16(wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5))
    A = dev_bf16(wl.normal_bf16(rng, (d_in, R), d_in ** -0.5))
    B = dev_bf16(wl.normal_bf16(rng, (R, d_out), R ** -0.5))
    offsets = np.array([0] + cuts + [T], np.int32)
    n = len(ranks)
    tab = dev_table(dict(offsets=offsets, rank=np.array(ranks, np.int32), scale=np.array(scales, np.float32),
                         flags=np.array([1] + [0] * (n - 1), np.int32), rung=np.zeros(n, np.int32), n_chunks=n))
    return X, W, A, B, tab, window


def test_matches_cwl_apply_on_two_calls_in_a_row():
    cases = [case(1, 300, 512, 320, 64, [70, 150, 260], [64, 8, 32, 16], [0.5, 4.0, 1.0, 2.0], 8),
             case(2, 130, 256, 128, 16, [40], [4, 16], [4.0, 1.0], 4)]
    expected = []
    for X, W, A, B, tab, window in cases:                     # the existing entry point, caller-owned workspace
        expected.append(y_to_f64(cwl.cwl_apply(X, W, A, B, tab, window)))
    torch.cuda.synchronize()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for (X, W, A, B, tab, window), want in zip(cases, expected):
        Y = torch.empty(X.shape[0], W.shape[1], dtype=torch.bfloat16, device="cuda")
        gc.collect()                                              # no garbage of earlier tests is freed during the call
        before = torch.cuda.memory_allocated()
        cwl.cwl_apply_noalloc(X, W, A, B, tab, window, Y, status_word=status)
        assert torch.cuda.memory_allocated() == before        # the call itself took nothing from the pool
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        check_output(y_to_f64(Y), want)                       # same kernel; only the order of fp32 sums may differ


def test_rejects_problems_larger_than_the_built_in_scratch():
    T, d_in, R = 16384, 1024, 256
    assert cwl.cwl_apply_noalloc_scratch_need(T, d_in, 256, R) > cwl.NOALLOC_SCRATCH_BYTES
    X = torch.zeros(T, d_in, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(d_in, 256, dtype=torch.bfloat16, device="cuda")
    A = torch.zeros(d_in, R, dtype=torch.bfloat16, device="cuda")
    B = torch.zeros(R, 256, dtype=torch.bfloat16, device="cuda")
    Y = torch.full((T, 256), 7.0, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(cwl.CwlError) as e:
        cwl.cwl_apply_noalloc(X, W, A, B, cwl.DeviceChunkTable(1), 0, Y)
    assert e.value.status == 5
    torch.cuda.synchronize()
    assert bool((Y == 7.0).all())                             # nothing was launched
