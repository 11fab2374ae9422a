"""GPU parity of cwl_apply_batch (several independent adapted projections, each with its own activations and shapes, in
one launch) against the fp64 oracle, element by element, through the C ABI; against guard bands; and against the
same projections issued one by one."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_output, dev_bf16, dev_table, host_table, status_ok, y_to_f64
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl
from test_gpu_apply import simple_table

pytestmark = pytest.mark.gpu


def make_items(seed, T, shapes, R):
    rng = np.random.default_rng(seed)
    host = []
    for d_in, d_out in shapes:
        host.append(dict(X=wl.normal_bf16(rng, (T, d_in), 1.0), W=wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5),
                         A=wl.normal_bf16(rng, (d_in, R), d_in ** -0.5), B=wl.normal_bf16(rng, (R, d_out), R ** -0.5)))
    dev = [{k: dev_bf16(v) for k, v in h.items()} for h in host]
    return host, dev


def guarded(T, d_out, extra_rows=3, extra_cols=16):
    buf = torch.full((T + extra_rows, d_out + extra_cols), float("nan"), dtype=torch.bfloat16, device="cuda")
    return buf, buf[:T, :d_out]


@pytest.mark.parametrize("T,shapes,R", [(200, [(512, 768), (1280, 384)], 32),                 # two items, different d_in
                                        (256, [(2048, 1536), (1024, 2048), (512, 320)], 64),   # three items, K splits
                                        (77, [(256, 256), (384, 528), (640, 128), (128, 1040)], 16)])
def test_matches_the_oracle_and_stays_inside_its_outputs(T, shapes, R):
    host, dev = make_items(T + len(shapes), T, shapes, R)
    cuts = list(range(29, T, 41))
    n = len(cuts) + 1
    ranks = ([R, R // 2, R // 4] * n)[:n]
    tab = simple_table(T, cuts, ranks, [float(R) / r for r in ranks], flags=[1] + [0] * (n - 1))   # scale = alpha / rank, alpha = R
    bufs = [guarded(T, d_out) for _, d_out in shapes]
    call = cwl.BatchCall([d["X"] for d in dev], [d["W"] for d in dev], [d["A"] for d in dev], [d["B"] for d in dev],
                         [y for _, y in bufs])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    call(dev_table(tab), 8, status_word=status)
    torch.cuda.synchronize()
    status_ok(status)
    for h, (buf, Y), (_, d_out) in zip(host, bufs, shapes):
        assert bool(torch.isnan(buf[T:, :]).all()) and bool(torch.isnan(buf[:, d_out:]).all())
        assert not bool(torch.isnan(Y).any())
        ref = oracle.apply(h["X"], h["W"], h["A"], h["B"], host_table(tab), 8)
        check_output(y_to_f64(Y.contiguous()), ref, label=f"batch item {h['W'].shape}")


def test_equals_separate_calls_with_row_gates_and_without_adapters():
    T, R, shapes = 130, 32, [(768, 512), (512, 1024)]
    host, dev = make_items(5, T, shapes, R)
    rng = np.random.default_rng(9)
    # row gates through the scheduler: a few steps of cwl_stream_step give every row a descriptor
    pol = cwl.make_policy([8, 16, 32], [4.0, 2.0, 1.0], [0.3, 0.7], 2, 6, 2)
    ds = cwl.DeviceStream(T, pol)
    for _ in range(5):
        ds.step(torch.from_numpy(rng.uniform(0, 1, T).astype(np.float32)).cuda())
    Ys = [torch.empty(T, d_out, dtype=torch.bfloat16, device="cuda") for _, d_out in shapes]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cwl.BatchCall([d["X"] for d in dev], [d["W"] for d in dev], [d["A"] for d in dev], [d["B"] for d in dev], Ys)(
        None, 0, gates=ds.gates, status_word=status)
    torch.cuda.synchronize()
    status_ok(status)
    for d, Y in zip(dev, Ys):
        want = cwl.cwl_apply_rows(d["X"], d["W"], d["A"], d["B"], ds.gates)
        assert float((Y.float() - want.float()).abs().max()) <= float(want.float().abs().max()) * 2.0 ** -7
    # no adapters: plain projections
    cwl.BatchCall([d["X"] for d in dev], [d["W"] for d in dev], None, None, Ys)(None, 0, status_word=status)
    torch.cuda.synchronize()
    status_ok(status)
    for h, Y in zip(host, Ys):
        check_output(y_to_f64(Y), oracle.apply(h["X"], h["W"], None, None, None, 0), label="batch dense")


def test_argument_errors():
    T, R = 32, 16
    host, dev = make_items(1, T, [(64, 64)], R)
    d = dev[0]
    Y = torch.empty(T, 64, dtype=torch.bfloat16, device="cuda")
    items = (cwl.CBatchItem * 1)(cwl.CBatchItem(d["X"].data_ptr(), 64, 64, d["W"].data_ptr(), 64, d["A"].data_ptr(), R,
                                                 d["B"].data_ptr(), 64, Y.data_ptr(), 64, 64))
    null_tab = cwl.CChunkTable(None, None, None, None, None, None, 0)
    L = cwl.lib()
    assert L.cwl_apply_batch(items, 0, T, R, null_tab, None, 0, None, 0, None, None) == 1       # n < 1
    assert L.cwl_apply_batch(items, 5, T, R, null_tab, None, 0, None, 0, None, None) == 1       # n > CWL_MAX_BATCH
    assert L.cwl_apply_batch(None, 1, T, R, null_tab, None, 0, None, 0, None, None) == 1
    assert L.cwl_apply_batch(items, 1, T, R, null_tab, None, 0, None, 0, None, None) == 1       # adapter without a table
    tab = dev_table(simple_table(T, [], [R], [1.0]))
    assert L.cwl_apply_batch(items, 1, T, R, tab.c_struct(), None, 0, None, 0, None, None) == 5  # no workspace
