"""GPU parity of cwl_apply_grouped: several adapted projections of the same rows in one launch
(Sec. III-F: q, k, v read one activation; gate and up another).  Each output is compared with the
fp64 oracle's adapted projection of that weight set, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_output, dev_bf16, dev_table, host_table, status_ok, y_to_f64
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def table_for(T, cuts, ranks, scales, flags=None):
    offsets = [0] + list(cuts) + [T]
    n = len(offsets) - 1
    return dict(offsets=np.array(offsets, np.int32), rank=np.array(ranks, np.int32), scale=np.array(scales, np.float32),
                flags=np.array(flags or [1] + [0] * (n - 1), np.int32), rung=np.zeros(n, np.int32), n_chunks=n)


def run_group(T, d_in, d_outs, R, table, window, seed, adapter=True):
    rng = np.random.default_rng(seed)
    X = wl.normal_bf16(rng, (T, d_in), 1.0)
    Ws = [wl.normal_bf16(rng, (d_in, d), d_in ** -0.5) for d in d_outs]
    As = [wl.normal_bf16(rng, (d_in, R), d_in ** -0.5) for _ in d_outs] if adapter else None
    Bs = [wl.normal_bf16(rng, (R, d), R ** -0.5) for d in d_outs] if adapter else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Ys = cwl.cwl_apply_grouped(dev_bf16(X), [dev_bf16(W) for W in Ws], [dev_bf16(A) for A in As] if adapter else None,
                               [dev_bf16(B) for B in Bs] if adapter else None, dev_table(table) if adapter else None,
                               window, status_word=status)
    torch.cuda.synchronize()
    status_ok(status)
    for j, d in enumerate(d_outs):
        ref = oracle.apply(X, Ws[j], As[j] if adapter else None, Bs[j] if adapter else None,
                           host_table(table) if adapter else None, window)
        check_output(y_to_f64(Ys[j]), ref)


def test_three_projections_with_ladder_and_windows():
    T = 333
    tab = table_for(T, [17, 64, 65, 200, 280], [8, 64, 16, 32, 64, 8], [4, 0.5, 2, 1, 0.5, 4], flags=[1, 0, 0, 1, 0, 0])
    run_group(T, 512, [320, 192, 336], 64, tab, 8, seed=31)


def test_two_projections_rank16_and_different_widths():
    T = 256
    tab = table_for(T, [40, 90, 170], [4, 16, 8, 0], [4.0, 1.0, 2.0, 0.0])
    run_group(T, 128, [1040, 64], 16, tab, 4, seed=32)


def test_four_projections_at_rank_128():
    T = 160
    tab = table_for(T, [50, 100], [128, 64, 16], [0.25, 0.5, 2.0])
    run_group(T, 256, [128, 144, 160, 176], 128, tab, 6, seed=33)


def test_three_projections_at_the_largest_rank_and_a_split_shrink():
    T = 200                                                    # d_in = 2048, small T: the shrink is split along d_in
    tab = table_for(T, [60, 130], [256, 96, 32], [0.125, 0.5, 1.0])
    run_group(T, 2048, [128, 64, 192], 256, tab, 8, seed=36)


def test_group_without_adapter():
    run_group(300, 208, [336, 528], 16, None, 0, seed=34, adapter=False)


def test_group_of_one_equals_cwl_apply():
    T, d_in, d_out, R = 200, 256, 256, 64
    rng = np.random.default_rng(35)
    X, W = dev_bf16(wl.normal_bf16(rng, (T, d_in), 1.0)), dev_bf16(wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5))
    A, B = dev_bf16(wl.normal_bf16(rng, (d_in, R), d_in ** -0.5)), dev_bf16(wl.normal_bf16(rng, (R, d_out), R ** -0.5))
    tab = dev_table(table_for(T, [77], [64, 16], [0.5, 2.0]))
    y1 = cwl.cwl_apply(X, W, A, B, tab, 8)
    (y2,) = cwl.cwl_apply_grouped(X, [W], [A], [B], tab, 8)
    torch.cuda.synchronize()
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))


def test_argument_errors():
    X = torch.zeros(8, 64, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    A = torch.zeros(64, 40, dtype=torch.bfloat16, device="cuda")
    B = torch.zeros(40, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(cwl.CwlError) as e:                    # the ladder's top rank must be a multiple of 16
        cwl.cwl_apply_grouped(X, [W] * 3, [A] * 3, [B] * 3, cwl.DeviceChunkTable(1), 0)
    assert e.value.status == 3
    with pytest.raises(cwl.CwlError) as e:                    # more projections than a group holds
        cwl.cwl_apply_grouped(X, [W] * 5, None, None, None, 0)
    assert e.value.status == 1
