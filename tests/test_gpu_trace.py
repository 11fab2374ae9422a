"""The device timeline of the test build (cwl_trace_set): the traced pair fills its slots in order, the output is the
one the oracle gives, and switching the trace off leaves later calls untouched."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_output, dev_bf16, dev_table, host_table, y_to_f64
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_a_traced_pair_records_an_ordered_timeline_and_the_result_is_unchanged():
    T, d_in, d_out, R = 256, 1024, 1536, 64
    rng = np.random.default_rng(77)
    X = wl.normal_bf16(rng, (T, d_in), 1.0); W = wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5)
    A = wl.normal_bf16(rng, (d_in, R), d_in ** -0.5); B = wl.normal_bf16(rng, (R, d_out), R ** -0.5)
    tab = dict(offsets=np.array([0, 100, T], np.int32), rank=np.array([64, 16], np.int32), scale=np.array([0.5, 2.0], np.float32),
               flags=np.array([1, 0], np.int32), rung=np.zeros(2, np.int32), n_chunks=2)
    args = (dev_bf16(X), dev_bf16(W), dev_bf16(A), dev_bf16(B), dev_table(tab), 8)
    ref = oracle.apply(X, W, A, B, host_table(tab), 8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    slots = torch.zeros(1024, dtype=torch.int64, device="cuda")
    with cwl.test_hooks() as L:
        L.cwl_trace_set.restype = C.c_int
        L.cwl_trace_set.argtypes = [C.c_void_p, C.c_int32]
        assert L.cwl_trace_set(slots.data_ptr(), 0) == 0
        Y = cwl.cwl_apply(*args, status_word=status)
        torch.cuda.synchronize()
        assert L.cwl_trace_set(None, -1) == 0
        t = slots.cpu().numpy()
        slots.zero_()
        Y2 = cwl.cwl_apply(*args, status_word=status)              # tracing off: nothing is written any more
        torch.cuda.synchronize()
        assert int(slots.abs().sum().item()) == 0
    assert int(status.item()) == 0
    check_output(y_to_f64(Y), ref, "traced call")
    assert torch.equal(Y, Y2)
    n = int((t[400:690] != 0).sum())
    assert n >= 4                                                   # pair 0 had work: K blocks of a shrink item, a tile, or both
    assert t[0] > 0 and t[0] <= t[1] <= t[400] and t[2] >= t[400 + n - 1] and t[4] >= t[3] >= t[5] >= t[2]
    issued, landed, committed = t[100:100 + n], t[400:400 + n], t[700:700 + n]
    assert (np.diff(landed) >= 0).all() and (issued <= landed).all() and (landed <= committed).all()


def test_the_read_probes_of_the_test_build_run_and_refuse_bad_arguments():
    region = torch.zeros(148 * 16384 * 4, dtype=torch.uint8, device="cuda")
    hot = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    with cwl.test_hooks() as L:
        L.cwl_probe_read.restype = C.c_int
        L.cwl_probe_read.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.cwl_probe_read_mix.restype = C.c_int
        L.cwl_probe_read_mix.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_uint32, C.c_int32, C.c_void_p, C.c_void_p]
        assert L.cwl_probe_read(region.data_ptr(), region.numel(), status.data_ptr(), stream) == 0
        for ctas, piece in ((148, 10752), (124, 16384), (1, 16)):
            assert L.cwl_probe_read_mix(region.data_ptr(), region.numel(), hot.data_ptr(), hot.numel(), piece, ctas,
                                        status.data_ptr(), stream) == 0
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        INVALID = 1
        assert L.cwl_probe_read(region.data_ptr(), 1000, status.data_ptr(), stream) == INVALID                  # too small
        assert L.cwl_probe_read_mix(region.data_ptr(), region.numel(), hot.data_ptr(), hot.numel(), 24, 148,
                                    status.data_ptr(), stream) == INVALID                                       # not a multiple of 16
        assert L.cwl_probe_read_mix(region.data_ptr(), region.numel(), hot.data_ptr(), hot.numel(), 4096, 149,
                                    status.data_ptr(), stream) == INVALID                                       # more CTAs than SMs
        assert L.cwl_probe_read_mix(region.data_ptr(), region.numel(), hot.data_ptr(), 64, 4096, 148,
                                    status.data_ptr(), stream) == INVALID                                       # hot region smaller than a piece
        assert L.cwl_probe_read_mix(region.data_ptr() + 16, region.numel() - 16, hot.data_ptr(), hot.numel(), 4096, 148,
                                    status.data_ptr(), stream) == INVALID                                       # unaligned
    torch.cuda.synchronize()
    assert int(status.item()) == 0
