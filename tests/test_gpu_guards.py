"""Nothing is written outside the outputs and nothing inside them is left unwritten.  Outputs sit in larger
buffers filled with a sentinel: guard rows after the last row and guard columns between d_out and the leading
dimension.  Afterwards every guard still holds the sentinel and no output element does.  Covered: whole-tile
epilogue with ragged edges, split-K epilogue, grouped launch, per-row gates, score and partition.  The workspace
is scratch in the full sense: whatever bytes it holds before a call, the outputs are the same."""
import numpy as np
import pytest
import torch

from gpu_util import dev_bf16, dev_table
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu
SENTINEL = float("nan")   # no finite input produces it, so an output element that still holds it was never written


def guarded(T, d_out, extra_rows=5, extra_cols=24):
    buf = torch.full((T + extra_rows, d_out + extra_cols), SENTINEL, dtype=torch.bfloat16, device="cuda")
    return buf, buf[:T, :d_out]


def check_guards(buf, T, d_out):
    assert bool(torch.isnan(buf[T:, :]).all()), "wrote below the last row"
    assert bool(torch.isnan(buf[:, d_out:]).all()), "wrote right of the last column"
    assert not bool(torch.isnan(buf[:T, :d_out]).any()), "left an output element unwritten"


def operands(seed, T, d_in, d_outs, R):
    rng = np.random.default_rng(seed)
    X = dev_bf16(wl.normal_bf16(rng, (T, d_in), 1.0))
    Ws = [dev_bf16(wl.normal_bf16(rng, (d_in, d), d_in ** -0.5)) for d in d_outs]
    As = [dev_bf16(wl.normal_bf16(rng, (d_in, R), d_in ** -0.5)) for _ in d_outs]
    Bs = [dev_bf16(wl.normal_bf16(rng, (R, d), R ** -0.5)) for d in d_outs]
    return X, Ws, As, Bs


def table(T, R):
    cuts = list(range(37, T, 53))
    n = len(cuts) + 1
    return dev_table(dict(offsets=np.array([0] + cuts + [T], np.int32), rank=np.array(([R, R // 2, R // 4] * n)[:n], np.int32),
                          scale=np.array(([1.0, 2.0, 4.0] * n)[:n], np.float32), flags=np.array([1] + [0] * (n - 1), np.int32),
                          rung=np.zeros(n, np.int32), n_chunks=n))


@pytest.mark.parametrize("T,d_in,d_out,R", [(300, 256, 336, 64),      # ragged rows and a ragged last column chunk
                                            (1000, 512, 1040, 16),    # several row tiles, widths 512 + 512 + 16
                                            (130, 2048, 528, 64),     # decode-sized: split-K epilogue
                                            (64, 4096, 4096, 64)])    # one partly filled row tile, split K
def test_cwl_apply_stays_inside_its_output(T, d_in, d_out, R):
    X, (W,), (A,), (B,) = operands(T, T, d_in, [d_out], R)
    buf, Y = guarded(T, d_out)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cwl.cwl_apply(X, W, A, B, table(T, R), 8, Y=Y, status_word=status)
    cwl.cwl_apply(X, W, None, None, None, 0, Y=Y, status_word=status)           # and the plain projection
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_guards(buf, T, d_out)


@pytest.mark.parametrize("fill", ["ones", "random", "stale"])
def test_workspace_contents_do_not_matter(fill):
    """The counters and flags in the workspace are tagged per launch, so nothing has to be cleared: bytes of any
    kind (all ones, random, or what earlier calls of other shapes left there) give bit-identical outputs."""
    shapes = [(300, 1024, 336, 64), (130, 2048, 528, 64), (64, 4096, 4096, 64), (700, 512, 1040, 16)]
    ws_bytes = max(cwl.cwl_apply_workspace_bytes(T, d_in, d_out, R) for T, d_in, d_out, R in shapes)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for rounds in range(2):
        for T, d_in, d_out, R in shapes:
            X, (W,), (A,), (B,) = operands(T + 1, T, d_in, [d_out], R)
            tab = table(T, R)
            ref = cwl.cwl_apply(X, W, A, B, tab, 8, workspace=torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda"),
                                status_word=status)
            if fill == "ones":
                ws.fill_(255)
            elif fill == "random":
                ws.copy_(torch.randint(0, 256, (ws_bytes,), dtype=torch.uint8, device="cuda"))
            got = cwl.cwl_apply(X, W, A, B, tab, 8, workspace=ws, status_word=status)      # "stale": left as it is
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert torch.equal(ref.view(torch.int16), got.view(torch.int16))


def test_grouped_and_per_row_calls_stay_inside_their_outputs():
    T, d_in, R = 700, 256, 32
    d_outs = [336, 512, 80]
    X, Ws, As, Bs = operands(9, T, d_in, d_outs, R)
    bufs = [guarded(T, d) for d in d_outs]
    cwl.cwl_apply_grouped(X, Ws, As, Bs, table(T, R), 4, Ys=[y for _, y in bufs])
    torch.cuda.synchronize()
    for (buf, _), d in zip(bufs, d_outs):
        check_guards(buf, T, d)
    gates = np.zeros(T, dtype=[("rank_in", np.int32), ("rank_out", np.int32), ("scale_in", np.float32), ("scale_out", np.float32),
                               ("lam", np.float32), ("pos_in_chunk", np.int32), ("opened", np.int32)])
    gates["rank_in"], gates["scale_in"], gates["lam"] = R, 1.0, 1.0
    g = torch.from_numpy(gates.view(np.uint8).reshape(T, -1)).cuda()
    buf, Y = guarded(T, d_outs[0])
    cwl.cwl_apply_rows(X, Ws[0], As[0], Bs[0], g, Y=Y)
    torch.cuda.synchronize()
    check_guards(buf, T, d_outs[0])


def test_score_and_partition_write_exactly_their_outputs():
    T, V = 777, 1001
    z = torch.randn(T + 3, V + 7, device="cuda")[:T, :V]                  # a strided view: rows are not contiguous
    score = torch.full((T + 8,), SENTINEL, device="cuda")
    cwl.cwl_score_tokens(z, score[:T])
    assert bool(torch.isnan(score[T:]).all()) and not bool(torch.isnan(score[:T]).any())
    pol = cwl.make_policy([4, 8, 16], [4.0, 2.0, 1.0], [0.9, 0.95], 8, 64, 4)
    cu = torch.tensor([0, 300, 300, T], dtype=torch.int32, device="cuda")
    tab = cwl.DeviceChunkTable(T // 8 + 4)
    for t in (tab.offsets, tab.rank, tab.rung, tab.flags):
        t.fill_(-99)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cwl.cwl_partition(score[:T].contiguous(), cu, pol, table=tab, status_word=status)
    n = int(tab.n_chunks.item())
    assert int(status.item()) == 0 and 0 < n <= tab.capacity
    assert bool((tab.offsets[n + 1:] == -99).all()) and bool((tab.rank[n:] == -99).all()) and bool((tab.flags[n:] == -99).all())
    assert int(tab.offsets[0]) == 0 and int(tab.offsets[n]) == T


@pytest.mark.parametrize("budget", [37, 26, 9, 1])
def test_a_call_planned_for_a_share_of_the_gpu_stays_inside_its_output_and_matches_the_full_plan(budget):
    # cwl_set_pair_budget changes the plan (tile widths, K split, who computes the shrink), never the result
    T, d_in, d_out, R = 200, 2048, 1552, 64
    X, (W,), (A,), (B,) = operands(77, T, d_in, [d_out], R)
    tab = table(T, R)
    want = cwl.cwl_apply(X, W, A, B, tab, 8)
    buf, Y = guarded(T, d_out)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    try:
        cwl.cwl_set_pair_budget(budget)
        cwl.cwl_apply(X, W, A, B, tab, 8, Y=Y, status_word=status)
    finally:
        cwl.cwl_set_pair_budget(0)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_guards(buf, T, d_out)
    # the same products summed in another order: fp32 rounding differences only, at most one bf16 ulp after rounding
    a, b = Y.float(), want.float()
    assert float((a - b).abs().max()) <= float(b.abs().max()) * 2.0 ** -7
    with pytest.raises(cwl.CwlError):
        cwl.cwl_set_pair_budget(-1)
