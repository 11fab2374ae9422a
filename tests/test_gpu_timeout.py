"""The failure path of cwl_apply without a device fault: with the test hook (test build of the library only) the
shrink never publishes H', every
wait on it runs out after a short limit, the kernel reports CWL_ERR_TIMEOUT in the status word and returns, and
the very next ordinary call on the same context is correct."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_output, dev_bf16, dev_table, host_table, y_to_f64
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu
CWL_ERR_TIMEOUT = 7


def test_withheld_publication_times_out_and_the_context_stays_usable():
    T, d_in, d_out, R = 300, 256, 320, 64
    rng = np.random.default_rng(41)
    X = wl.normal_bf16(rng, (T, d_in), 1.0); W = wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5)
    A = wl.normal_bf16(rng, (d_in, R), d_in ** -0.5); B = wl.normal_bf16(rng, (R, d_out), R ** -0.5)
    tab = dict(offsets=np.array([0, 120, T], np.int32), rank=np.array([64, 16], np.int32), scale=np.array([0.5, 2.0], np.float32),
               flags=np.array([1, 0], np.int32), rung=np.zeros(2, np.int32), n_chunks=2)
    args = (dev_bf16(X), dev_bf16(W), dev_bf16(A), dev_bf16(B), dev_table(tab), 8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with cwl.test_hooks():                                                       # the test build of the library
        cwl.cwl_debug_set(wait_limit_ns=20_000_000, withhold_publish=True)      # 20 ms
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        cwl.cwl_apply(*args, status_word=status)
        end.record()
        torch.cuda.synchronize()                                                 # returns: nothing hangs
        assert int(status.item()) & (1 << CWL_ERR_TIMEOUT)
        assert start.elapsed_time(end) < 2000.0                                  # a few wait limits, not seconds
    status.zero_()
    Y = cwl.cwl_apply(*args, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_output(y_to_f64(Y), oracle.apply(X, W, A, B, host_table(tab), 8))
