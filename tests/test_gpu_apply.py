"""GPU parity of cwl_apply (adapted projection, Sec. III-F, with the cross-fade of Sec. III-D)
against the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_output, dev_bf16, dev_table, host_table, status_ok, table_dict, y_to_f64
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run_case(T, d_in, d_out, R, table, window, seed, adapter=True):
    rng = np.random.default_rng(seed)
    X = wl.normal_bf16(rng, (T, d_in), 1.0)
    W = wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5)
    A = wl.normal_bf16(rng, (d_in, R), d_in ** -0.5) if adapter else None
    B = wl.normal_bf16(rng, (R, d_out), R ** -0.5) if adapter else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = cwl.cwl_apply(dev_bf16(X), dev_bf16(W), dev_bf16(A) if adapter else None, dev_bf16(B) if adapter else None,
                      dev_table(table) if adapter else None, window, status_word=status)
    torch.cuda.synchronize()
    status_ok(status)
    ref = oracle.apply(X, W, A, B, host_table(table) if adapter else None, window)
    return check_output(y_to_f64(Y), ref)


def simple_table(T, cuts, ranks, scales, flags=None):
    offsets = [0] + list(cuts) + [T]
    n = len(offsets) - 1
    return dict(offsets=np.array(offsets, np.int32), rank=np.array(ranks, np.int32),
                scale=np.array(scales, np.float32), flags=np.array(flags or [1] + [0] * (n - 1), np.int32),
                rung=np.zeros(n, np.int32), n_chunks=n)


def test_dense_base_only_one_tile():
    run_case(128, 64, 256, 16, None, 0, seed=1, adapter=False)


def test_dense_base_multi_tile_ragged():
    # 3 row tiles with a ragged tail, K not a multiple of 64, N spanning two column tiles with a ragged tail
    run_case(300, 208, 336, 16, None, 0, seed=2, adapter=False)


def test_full_rank_single_chunk():
    T = 200
    run_case(T, 256, 256, 64, simple_table(T, [], [64], [0.5]), 8, seed=3)


def test_rank16_ladder_with_windows():
    T = 256
    tab = simple_table(T, [40, 90, 170], [4, 16, 8, 0], [4.0, 1.0, 2.0, 0.0])
    run_case(T, 128, 192, 16, tab, 4, seed=4)


def test_mixed_sequences_and_ranks_R64():
    T = 333
    tab = simple_table(T, [17, 64, 65, 200, 280], [8, 64, 16, 32, 64, 8], [4, 0.5, 2, 1, 0.5, 4],
                       flags=[1, 0, 0, 1, 0, 0])
    run_case(T, 512, 320, 64, tab, 8, seed=5)


@pytest.mark.parametrize("R", [32, 128, 256])
def test_other_max_ranks(R):
    T = 160
    tab = simple_table(T, [50, 100], [R, R // 2, 16], [32.0 / R, 64.0 / R, 2.0])
    run_case(T, 256, 128, R, tab, 6, seed=6 + R)


def test_rows_outside_the_table_get_no_adapter():
    T = 64
    rng = np.random.default_rng(11)
    X = wl.normal_bf16(rng, (T, 64), 1.0)
    W = wl.normal_bf16(rng, (64, 64), 0.125)
    A = wl.normal_bf16(rng, (64, 16), 0.125)
    B = wl.normal_bf16(rng, (16, 64), 0.25)
    empty = cwl.DeviceChunkTable(4)
    Y = cwl.cwl_apply(dev_bf16(X), dev_bf16(W), dev_bf16(A), dev_bf16(B), empty, 4)
    check_output(y_to_f64(Y), oracle.apply(X, W, None, None, None, 0))


def test_config1_full_output():
    w = wl.config1()
    p = w.policy
    tab = oracle.partition(w.score, w.cu_seqlens, p.ranks, p.scales, p.thresholds, p.min_len, p.max_len, p.window)
    pr = w.projections[0]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = cwl.cwl_apply(dev_bf16(w.X[1024]), dev_bf16(pr.W), dev_bf16(pr.A), dev_bf16(pr.B),
                      dev_table(table_dict(tab)), p.window, status_word=status)
    torch.cuda.synchronize()
    status_ok(status)
    res = check_output(y_to_f64(Y), oracle.apply(w.X[1024], pr.W, pr.A, pr.B, tab, p.window))
    assert res["rel_fro"] < 5e-3


def test_static_lora_and_decode_tables_small():
    # static full-rank LoRA = one chunk per sequence; decode = one first-of-sequence chunk per row
    T = 96
    run_case(T, 128, 128, 64, wl.static_table(np.array([0, 40, 96]), 64, 32.0), 8, seed=20)
    w4 = wl.config4(T=T)
    run_case(T, 128, 128, 64, w4.table, 0, seed=21)


def test_split_k_with_partials_too_large_to_land():
    """Decode-sized rows against a large projection: 512-wide tiles whose K loop is split 3-way.  The two other
    contributors' partial sums of a CTA's share (2 x 88 KB) do not fit the operand ring beside the staged rows,
    so the hand-over reads them from global memory instead of landing them by bulk copies."""
    T, d_in, d_out = 8, 11008, 11008
    plan = cwl.cwl_apply_plan(T, d_in, d_out, 64)
    assert plan["split_k"] == 3 and plan["wide_width"] == 512
    w4 = wl.config4(T=T)
    run_case(T, d_in, d_out, 64, w4.table, 0, seed=22)
    run_case(T, d_in, d_out, 64, None, 0, seed=23, adapter=False)


def test_argument_errors():
    X = torch.zeros(8, 64, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    A = torch.zeros(64, 24, dtype=torch.bfloat16, device="cuda")
    B = torch.zeros(24, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(cwl.CwlError) as e:
        cwl.cwl_apply(X, W, A, B, cwl.DeviceChunkTable(1), 0)            # R = 24 is not a multiple of 16
    assert e.value.status == 3
    A = torch.zeros(64, 16, dtype=torch.bfloat16, device="cuda")
    B = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(cwl.CwlError) as e:
        cwl.cwl_apply(X, W, A, B, cwl.DeviceChunkTable(1), 0, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 5
    assert cwl.cwl_apply(X[:0], W, A, B, cwl.DeviceChunkTable(1), 0).shape == (0, 64)


def test_many_row_tiles_and_widest_rank():
    # 1300 row tiles of 256 (far more than one wave) on a narrow projection, R = 256: the item loop, the shrink
    # hand-out and the per-tile flags at scale; sampled rows against the oracle
    T, d_in, d_out, R = 332_801, 64, 96, 256
    rng = np.random.default_rng(77)
    X = wl.normal_bf16(rng, (T, d_in), 1.0)
    W = wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5)
    A = wl.normal_bf16(rng, (d_in, R), d_in ** -0.5)
    B = wl.normal_bf16(rng, (R, d_out), R ** -0.5)
    cuts = list(range(1000, T, 1000))
    n = len(cuts) + 1
    tab = simple_table(T, cuts, ([256, 64, 0, 128] * n)[:n], ([0.125, 0.5, 0.0, 0.25] * n)[:n], flags=([1, 0, 0, 0, 0] * n)[:n])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = cwl.cwl_apply(dev_bf16(X), dev_bf16(W), dev_bf16(A), dev_bf16(B), dev_table(tab), 8, status_word=status)
    torch.cuda.synchronize()
    status_ok(status)
    rows = np.unique(np.concatenate([[0, 255, 256, T - 2, T - 1], rng.integers(0, T, 200),
                                     np.array(cuts[:40]), np.array(cuts[:40]) + 3])).astype(np.int32)
    ref = oracle.apply(X, W, A, B, host_table(tab), 8, rows=rows)
    check_output(y_to_f64(Y[torch.from_numpy(rows.astype(np.int64)).cuda()]), ref)


def test_single_row_and_tiny_widths():
    run_case(1, 16, 16, 16, simple_table(1, [], [16], [1.0]), 0, seed=78)
    run_case(5, 48, 32, 32, simple_table(5, [2], [32, 16], [1.0, 2.0]), 2, seed=79)
