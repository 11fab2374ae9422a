"""GPU parity of cwl_apply_mode with the centred cross-fade window (Sec. III-D variant: the window lies around the
join) against the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_output, dev_bf16, dev_table, host_table, status_ok, y_to_f64
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl
from test_gpu_apply import simple_table

pytestmark = pytest.mark.gpu


def run_centred(T, d_in, d_out, R, table, window, seed):
    rng = np.random.default_rng(seed)
    X = wl.normal_bf16(rng, (T, d_in), 1.0)
    W = wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5)
    A = wl.normal_bf16(rng, (d_in, R), d_in ** -0.5)
    B = wl.normal_bf16(rng, (R, d_out), R ** -0.5)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = cwl.cwl_apply(dev_bf16(X), dev_bf16(W), dev_bf16(A), dev_bf16(B), dev_table(table), window,
                      status_word=status, centred=True)
    torch.cuda.synchronize()
    status_ok(status)
    ref = oracle.apply(X, W, A, B, host_table(table), window, centred=True)
    check_output(y_to_f64(Y), ref, label=f"centred window {window}")
    return y_to_f64(Y), (X, W, A, B)


@pytest.mark.parametrize("window", [0, 1, 2, 5, 8])
def test_windows_around_joins_of_mixed_sequences(window):
    T = 333
    tab = simple_table(T, [17, 64, 80, 200, 280], [8, 64, 16, 32, 64, 8], [4, 0.5, 2, 1, 0.5, 4],
                       flags=[1, 0, 0, 1, 0, 0])
    run_centred(T, 512, 320, 64, tab, window, seed=50 + window)


def test_window_rows_differ_from_the_causal_placement_only_around_joins():
    T = 256
    tab = simple_table(T, [100, 180], [4, 16, 8], [4.0, 1.0, 2.0])
    Yc, (X, W, A, B) = run_centred(T, 128, 192, 16, tab, 6, seed=61)
    Yk = y_to_f64(cwl.cwl_apply(dev_bf16(X), dev_bf16(W), dev_bf16(A), dev_bf16(B), dev_table(tab), 6))
    same = np.all(Yc == Yk, axis=1)
    touched = set(range(97, 106)) | set(range(177, 186))        # rows of either placement's window at the two joins
    assert all(same[t] for t in range(T) if t not in touched)
    assert not all(same[t] for t in touched)


def test_short_chunks_and_a_window_split_by_a_row_tile_edge():
    # the join at row 128 sits on the edge between two 128-row tiles: its window spans both; chunk [128, 131) is
    # shorter than the window, so its rows are claimed by the join that opens it first
    T = 300
    tab = simple_table(T, [128, 131, 250], [16, 4, 8, 16], [1.0, 4.0, 2.0, 1.0])
    run_centred(T, 128, 128, 16, tab, 6, seed=62)


def test_unknown_mode_is_rejected():
    X = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    Y = torch.empty(16, 64, dtype=torch.bfloat16, device="cuda")
    null_tab = cwl.CChunkTable(None, None, None, None, None, None, 0)
    rc = cwl.lib().cwl_apply_mode(X.data_ptr(), 64, W.data_ptr(), 64, None, 0, None, 0, 16, 64, 64, 0, null_tab, 0, 7,
                                  Y.data_ptr(), 64, None, 0, None, None)
    assert rc == 1
