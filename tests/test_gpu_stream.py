"""GPU parity of the decode-time scheduler (cwl_stream_*, Sec. III-B: tokens grouped as they arrive, state kept from step
to step) and of the per-row adapted projection cwl_apply_rows, against the oracle, through the C ABI.
Gates are integer decisions plus copied scales and an fp32 quotient: compared bit by bit."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_output, dev_bf16, status_ok, y_to_f64
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu
FIELDS = ("rank_in", "rank_out", "scale_in", "scale_out", "lam", "pos_in_chunk", "opened")


def assert_gates_equal(got, ref_list, active=None):
    for n, ref in enumerate(ref_list):
        if active is not None and not active[n]:
            assert got[n]["rank_in"] == 0 and got[n]["pos_in_chunk"] == -1 and got[n]["lam"] == 1.0
            continue
        for f in FIELDS:
            assert got[n][f].tobytes() == ref[f].tobytes(), (n, f, got[n][f], ref[f])


@pytest.mark.parametrize("seed", range(6))
def test_many_sequences_many_steps_bit_exact(seed):
    rng = np.random.default_rng(700 + seed)
    n_seq = int(rng.choice([1, 37, 257]))
    min_len = int(rng.integers(1, 17))
    max_len = min_len * int(rng.integers(1, 5))
    window = int(rng.integers(0, min_len + 1))
    hi_budget = int(rng.choice([-1, 0, 2]))
    ranks, scales, ths = [8, 16, 32, 64], [4.0, 2.0, 1.0, 0.5], [0.25, 0.5, 0.75]
    pol = cwl.make_policy(ranks, scales, ths, min_len, max_len, window, hi_budget)
    ds = cwl.DeviceStream(n_seq, pol)
    refs = [oracle.Stream(ranks, scales, ths, min_len, max_len, window, hi_budget) for _ in range(n_seq)]
    level = rng.uniform(0, 1, size=n_seq)
    for step in range(120):
        if step % 15 == 0:
            level = rng.uniform(0, 1, size=n_seq)                       # regime switches
        s = np.clip(level + rng.normal(0, 0.07, n_seq), -0.1, 1.1).astype(np.float32)
        if step == 40:
            s[0] = np.nan                                               # NaN counts as hardest
        active = (rng.uniform(size=n_seq) < 0.9).astype(np.int32) if seed % 2 else None
        ds.step(torch.from_numpy(s).cuda(), torch.from_numpy(active).cuda() if active is not None else None)
        got = ds.gates_to_host()
        ref = [refs[n].step(s[n]) if (active is None or active[n]) else None for n in range(n_seq)]
        assert_gates_equal(got, ref, active)


def test_reset_starts_sequences_over():
    pol = cwl.make_policy([4, 16], [4.0, 1.0], [0.5], 2, 4, 1)
    ds = cwl.DeviceStream(3, pol)
    s = torch.tensor([0.9, 0.1, 0.9], device="cuda")
    for _ in range(5):
        ds.step(s)
    ds.reset()
    ds.step(s)
    g = ds.gates_to_host()
    assert (g["opened"] == 1).all() and (g["pos_in_chunk"] == 0).all() and (g["lam"] == 1.0).all()
    assert g["rank_in"].tolist() == [16, 4, 16]


def test_bad_arguments():
    with pytest.raises(cwl.CwlError):
        cwl.DeviceStream(4, cwl.make_policy([4, 16], [4.0, 1.0], [0.5], 65, 130, 0))    # min_len above the limit
    pol = cwl.make_policy([4, 16], [4.0, 1.0], [0.5], 2, 4, 1)
    ds = cwl.DeviceStream(4, pol)
    ds.state = torch.empty(8, dtype=torch.uint8, device="cuda")
    with pytest.raises(cwl.CwlError) as e:
        ds.step(torch.zeros(4, device="cuda"))
    assert e.value.status == 5


def gates_tensor(g: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(g).view(np.uint8).reshape(len(g), -1)).cuda()


def random_gates(rng, T, ladder, window):
    g = np.zeros(T, dtype=oracle.ROW_GATE_DTYPE)
    for t in range(T):
        r = int(rng.choice(ladder))
        g[t]["rank_in"], g[t]["scale_in"], g[t]["lam"] = r, np.float32(32.0 / r) if r else 0.0, 1.0
        if window and rng.uniform() < 0.4:
            j = int(rng.integers(0, window))
            r2 = int(rng.choice(ladder))
            g[t]["lam"] = np.float32(j + 1) / np.float32(window + 1)
            g[t]["rank_out"], g[t]["scale_out"], g[t]["pos_in_chunk"] = r2, np.float32(32.0 / r2) if r2 else 0.0, j
    return g


@pytest.mark.parametrize("T,d_in,d_out,R", [(96, 128, 192, 16), (256, 512, 1040, 64), (300, 256, 320, 64)])
def test_apply_rows_small(T, d_in, d_out, R):
    rng = np.random.default_rng(T + d_out)
    X = wl.normal_bf16(rng, (T, d_in), 1.0); W = wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5)
    A = wl.normal_bf16(rng, (d_in, R), d_in ** -0.5); B = wl.normal_bf16(rng, (R, d_out), R ** -0.5)
    g = random_gates(rng, T, [0, R // 4, R // 2, R], 8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = cwl.cwl_apply_rows(dev_bf16(X), dev_bf16(W), dev_bf16(A), dev_bf16(B), gates_tensor(g), status_word=status)
    torch.cuda.synchronize()
    status_ok(status)
    check_output(y_to_f64(Y), oracle.apply_rows(X, W, A, B, g))


def test_decode_loop_scheduler_feeds_apply_at_full_decode_size():
    # 256 sequences, one token each per step: scheduler -> per-row adapted projection 4096 -> 11008, every row checked
    w = wl.config4()
    pol = cwl.make_policy([8, 16, 32, 64], [4.0, 2.0, 1.0, 0.5], [0.25, 0.5, 0.75], 4, 16, 4)
    ds = cwl.DeviceStream(w.T, pol)
    refs = [oracle.Stream([8, 16, 32, 64], [4.0, 2.0, 1.0, 0.5], [0.25, 0.5, 0.75], 4, 16, 4) for _ in range(w.T)]
    rng = np.random.default_rng(9)
    pr = w.projections[0]
    X, W, A, B = dev_bf16(w.X[pr.d_in]), dev_bf16(pr.W), dev_bf16(pr.A), dev_bf16(pr.B)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for step in range(9):                                   # past the first joins, so some rows are inside a window
        s = rng.uniform(0, 1, w.T).astype(np.float32) if step % 4 == 0 else s
        gates = ds.step(torch.from_numpy(s).cuda())
        Y = cwl.cwl_apply_rows(X, W, A, B, gates, status_word=status)
        ref_g = np.array([r.step(x) for r, x in zip(refs, s)], dtype=oracle.ROW_GATE_DTYPE)
    torch.cuda.synchronize()
    status_ok(status)
    assert (ref_g["lam"] < 1.0).any()
    assert_gates_equal(ds.gates_to_host(), list(ref_g))
    check_output(y_to_f64(Y), oracle.apply_rows(w.X[pr.d_in], pr.W, pr.A, pr.B, ref_g))
