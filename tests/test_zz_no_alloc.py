"""cwl_apply_noalloc: the variant of the adapted projection for callers that cannot allocate device
memory (its scratch is a fixed array inside the library).  Collected last on purpose.

Checked through the C ABI against the ordinary cwl_apply AND against the fp64 oracle on the same
inputs, on two calls in a row with different shapes and tables, so that whatever the first call
leaves in the shared scratch must not leak into the second.  That the call allocates nothing is
read from the driver's free-memory figure (which sees any allocation made inside the library, not
just those of the tensor pool) around a call made after a warm-up call has loaded the kernels and
looked the scratch array's address up."""
import gc

import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_output, dev_bf16, dev_table, host_table, y_to_f64
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def case(seed, T, d_in, d_out, R, cuts, ranks, scales, window):
    rng = np.random.default_rng(seed)
    host = dict(X=wl.normal_bf16(rng, (T, d_in), 1.0), W=wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5),
                A=wl.normal_bf16(rng, (d_in, R), d_in ** -0.5), B=wl.normal_bf16(rng, (R, d_out), R ** -0.5))
    offsets = np.array([0] + cuts + [T], np.int32)
    n = len(ranks)
    tab = dict(offsets=offsets, rank=np.array(ranks, np.int32), scale=np.array(scales, np.float32),
               flags=np.array([1] + [0] * (n - 1), np.int32), rung=np.zeros(n, np.int32), n_chunks=n)
    dev = {k: dev_bf16(v) for k, v in host.items()}
    return host, dev, tab, window


def test_matches_cwl_apply_and_the_oracle_on_two_calls_in_a_row():
    cases = [case(1, 300, 512, 320, 64, [70, 150, 260], [64, 8, 32, 16], [0.5, 4.0, 1.0, 2.0], 8),
             case(2, 130, 256, 128, 16, [40], [4, 16], [4.0, 1.0], 4)]
    expected, reference, tables = [], [], []
    for host, dev, tab, window in cases:
        tables.append(dev_table(tab))
        # the existing entry point, caller-owned workspace, and the fp64 oracle
        expected.append(y_to_f64(cwl.cwl_apply(dev["X"], dev["W"], dev["A"], dev["B"], tables[-1], window)))
        reference.append(oracle.apply(host["X"], host["W"], host["A"], host["B"], host_table(tab), window))
    torch.cuda.synchronize()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    outs = [torch.empty(h["X"].shape[0], h["W"].shape[1], dtype=torch.bfloat16, device="cuda") for h, _, _, _ in cases]
    # warm-up call: loads the kernels and resolves the scratch array's address (documented as a first-call cost)
    _, dev, _, window = cases[0]
    cwl.cwl_apply_noalloc(dev["X"], dev["W"], dev["A"], dev["B"], tables[0], window, outs[0], status_word=status)
    torch.cuda.synchronize()
    for (host, dev, tab, window), dtab, Y, want, ref in zip(cases, tables, outs, expected, reference):
        Y.fill_(7.0)
        gc.collect()                                          # no garbage of earlier tests is freed during the call
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]            # the driver's figure: sees allocations of any origin
        pool_before = torch.cuda.memory_allocated()
        cwl.cwl_apply_noalloc(dev["X"], dev["W"], dev["A"], dev["B"], dtab, window, Y, status_word=status)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before    # nothing was taken from the device ...
        assert torch.cuda.memory_allocated() == pool_before   # ... nor from the tensor pool
        assert int(status.item()) == 0
        check_output(y_to_f64(Y), want, label="noalloc vs cwl_apply")    # same kernel; only the order of fp32 sums may differ
        check_output(y_to_f64(Y), ref, label="noalloc vs oracle")


@pytest.mark.parametrize("R", [24, 272])
def test_reports_an_unsupported_rank_as_cwl_apply_does(R):
    T, d = 64, 128
    X = torch.zeros(T, d, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(d, d, dtype=torch.bfloat16, device="cuda")
    A = torch.zeros(d, R, dtype=torch.bfloat16, device="cuda")
    B = torch.zeros(R, d, dtype=torch.bfloat16, device="cuda")
    Y = torch.empty(T, d, dtype=torch.bfloat16, device="cuda")
    tab = cwl.DeviceChunkTable(1)
    with pytest.raises(cwl.CwlError) as e:
        cwl.cwl_apply_noalloc(X, W, A, B, tab, 0, Y)
    assert e.value.status == 3                                # CWL_ERR_UNSUPPORTED, as cwl_apply reports it
    with pytest.raises(cwl.CwlError) as e2:
        cwl.cwl_apply(X, W, A, B, tab, 0, Y=Y, workspace=torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
    assert e2.value.status == 3


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
