"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times (HotPath: the
library's own workspaces, one stream, no host synchronisation between the calls).

The fp64 oracle cannot compute whole outputs at these sizes in test time, so rows are sampled and
compared one by one over all output columns: random rows, every window row of a few chunk joins,
first and last rows of a few chunks, the first and the last row.  Scores are compared on sampled
rows too; the chunk table is compared whole and bit by bit (given the GPU's fp32 scores)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_output, check_scores, y_to_f64
from paper_2601_21109_b200 import workloads as wl
from paper_2601_21109_b200.runner import HotPath

pytestmark = pytest.mark.gpu


def oracle_table(w, score, thresholds=None):
    p = w.policy
    return oracle.partition(score, w.cu_seqlens, p.ranks, p.scales, thresholds or p.thresholds, p.min_len, p.max_len,
                            p.window, p.hi_budget)


def assert_table_equal(got: dict, ref: oracle.ChunkTable):
    assert got["n_chunks"] == ref.n_chunks
    n = ref.n_chunks
    assert np.array_equal(got["offsets"], ref.offsets[:n + 1])
    assert np.array_equal(got["rank"], ref.rank[:n])
    assert np.array_equal(got["rung"], ref.rung[:n])
    assert np.array_equal(got["flags"] & 1, ref.flags[:n] & 1)
    assert np.array_equal(got["scale"].view(np.uint32), ref.scale[:n].view(np.uint32))


def check_projections(w, hp, tab, rows, window):
    worst = 0.0
    for dp, gp in zip(w.projections, hp.projs):
        ref = oracle.apply(w.X[dp.d_in], dp.W, dp.A, dp.B, tab, window, rows=rows)
        got = y_to_f64(gp.Y[torch.from_numpy(rows.astype(np.int64)).cuda()])
        res = check_output(got, ref, label=f"{w.name} {dp.name} T={w.T}", max_saved_frac=2e-4)
        worst = max(worst, res["rel_fro"])
    return worst


def scored_pipeline(w, n_score_rows, n_random, n_joins, n_edges):
    hp = HotPath(w)
    hp.score_step()
    s_gpu = hp.score.cpu().numpy()
    rng = np.random.default_rng(7)
    srows = np.unique(np.concatenate([[0, w.T - 1], rng.integers(0, w.T, n_score_rows)]))
    s_ref = oracle.score_tokens(w.logits[srows])
    check_scores(s_gpu[srows], s_ref, label=f"{w.name} scores, sampled rows")
    ths = np.percentile(s_gpu, [25, 50, 75]).astype(np.float32).tolist()   # rule-based percentile mapping (Sec. IV-C)
    hp.set_thresholds(ths)
    hp.step()
    torch.cuda.synchronize()
    assert int(hp.status.item()) == 0
    tab = oracle_table(w, s_gpu, hp.policy.thresholds)
    assert_table_equal(hp.table.to_host(), tab)
    rows = wl.sample_rows(rng, w.T, tab.offsets[:tab.n_chunks + 1], tab.flags, w.policy.window,
                          n_random=n_random, n_joins=n_joins, n_chunks_edges=n_edges)
    rel = check_projections(w, hp, tab, rows, w.policy.window)
    assert rel < 5e-3
    return tab


def test_config2_prefill_all_seven_projections():
    w = wl.config2()
    tab = scored_pipeline(w, n_score_rows=96, n_random=64, n_joins=8, n_edges=8)
    assert sorted(set(tab.rank[:tab.n_chunks].tolist())) == [8, 16, 32, 64]     # the whole ladder is exercised


def test_config3_packed_ragged_batch():
    w = wl.config3()
    hp = HotPath(w)
    hp.step()
    torch.cuda.synchronize()
    assert int(hp.status.item()) == 0
    tab = oracle_table(w, w.score)
    got = hp.table.to_host()
    assert_table_equal(got, tab)
    # chunks never cross a sequence boundary: every cu_seqlens entry is a chunk offset flagged first-of-sequence
    first = set(got["offsets"][:-1][(got["flags"] & 1) == 1].tolist())
    assert set(w.cu_seqlens[:-1].tolist()) <= first
    rng = np.random.default_rng(3)
    rows = wl.sample_rows(rng, w.T, tab.offsets[:tab.n_chunks + 1], tab.flags, w.policy.window, 64, 8, 8)
    ragged_tail = np.arange(max(0, w.T - 3), w.T, dtype=np.int32)      # the last, partly filled row tile
    rows = np.unique(np.concatenate([rows, ragged_tail, w.cu_seqlens[1:-1], w.cu_seqlens[1:-1] - 1])).astype(np.int32)
    assert check_projections(w, hp, tab, rows, w.policy.window) < 5e-3


def test_config4_decode_every_row():
    w = wl.config4()
    hp = HotPath(w)
    hp.step()
    torch.cuda.synchronize()
    assert int(hp.status.item()) == 0
    t = w.table
    tab = oracle.ChunkTable(t["offsets"], t["rank"], t["scale"], t["rung"], t["flags"], t["n_chunks"])
    rows = np.arange(w.T, dtype=np.int32)
    assert check_projections(w, hp, tab, rows, 0) < 5e-3


def test_config5_one_layer_of_the_stack():
    w = wl.config5_layer()
    scored_pipeline(w, n_score_rows=48, n_random=24, n_joins=4, n_edges=4)
    # the comparison runs through the same kernels: static full-rank LoRA and the dense floor, sampled rows
    hp = HotPath(w)
    st = wl.static_table(w.cu_seqlens, w.R, 32.0)
    from paper_2601_21109_b200 import binding as cwl
    static_tab = cwl.DeviceChunkTable.from_host(st["offsets"], st["rank"], st["scale"], st["flags"], st["rung"])
    rows = np.unique(np.concatenate([[0, w.T - 1], np.random.default_rng(5).integers(0, w.T, 12),
                                     w.cu_seqlens[1:-1], w.cu_seqlens[1:-1] - 1])).astype(np.int32)
    host_static = oracle.ChunkTable(st["offsets"], st["rank"], st["scale"], st["rung"], st["flags"], st["n_chunks"])
    hp.apply_step(table=static_tab)
    torch.cuda.synchronize()
    assert check_projections(w, hp, host_static, rows, w.policy.window) < 5e-3
    hp.apply_step(dense=True)
    torch.cuda.synchronize()
    for dp, gp in zip(w.projections, hp.projs):
        ref = oracle.apply(w.X[dp.d_in], dp.W, None, None, None, 0, rows=rows)
        check_output(y_to_f64(gp.Y[torch.from_numpy(rows.astype(np.int64)).cuda()]), ref)
    assert int(hp.status.item()) == 0
