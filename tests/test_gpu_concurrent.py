"""Two cwl_apply calls in flight at once on two streams with distinct workspaces, each large enough to want most
of the GPU for itself (its flags and counters only make progress once all its CTA pairs are resident).  Run
through the test build with a short device-side wait limit, so that the worst outcome is a CWL_ERR_TIMEOUT
status, never a hang.  Both outputs are checked against the oracle on sampled rows."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import check_output, dev_bf16, dev_table, host_table, y_to_f64
from paper_2601_21109_b200 import binding as cwl
from paper_2601_21109_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def problem(seed, T, d_in, d_out, R):
    rng = np.random.default_rng(seed)
    host = dict(X=wl.normal_bf16(rng, (T, d_in), 1.0), W=wl.normal_bf16(rng, (d_in, d_out), d_in ** -0.5),
                A=wl.normal_bf16(rng, (d_in, R), d_in ** -0.5), B=wl.normal_bf16(rng, (R, d_out), R ** -0.5))
    cuts = sorted(rng.choice(np.arange(64, T - 64, 16), size=5, replace=False).tolist())
    n = len(cuts) + 1
    rank = rng.choice([8, 16, 32, 64], n).astype(np.int32)
    # scale = alpha / rank as the ladder sets it: the gated shrink output is a bf16 tensor-core operand, so its rounding
    # (2^-9 relative) scales with the adapter term, which a large scale on a large rank would blow up beyond the 3e-2 gate
    tab = dict(offsets=np.array([0] + cuts + [T], np.int32), rank=rank, scale=(32.0 / rank).astype(np.float32),
               flags=np.array([1] + [0] * (n - 1), np.int32), rung=np.zeros(n, np.int32), n_chunks=n)
    return host, tab


@pytest.mark.parametrize("shapes", [((4096, 1024, 2048), (4096, 1024, 2048)),       # two prefill launches of 64 tiles each
                                    ((256, 2048, 4096), (3072, 512, 1536)),         # a split-K decode launch beside a prefill one
                                    ((256, 4096, 2048), (256, 2048, 4096))])        # two split-K launches
def test_two_streams_two_workspaces(shapes):
    R, window = 64, 8
    probs = [problem(70 + i, *shp, R) for i, shp in enumerate(shapes)]
    dev = [({k: dev_bf16(v) for k, v in h.items()}, dev_table(t)) for h, t in probs]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    status = [torch.zeros(1, dtype=torch.int32, device="cuda") for _ in range(2)]
    ws = [torch.empty(cwl.cwl_apply_workspace_bytes(*shp, R), dtype=torch.uint8, device="cuda") for shp in shapes]
    Y = [torch.empty(shp[0], shp[2], dtype=torch.bfloat16, device="cuda") for shp in shapes]
    torch.cuda.synchronize()
    with cwl.test_hooks():
        cwl.cwl_debug_set(wait_limit_ns=50_000_000)                  # 50 ms: a stuck wait ends as a status, quickly
        for rep in range(6):                                         # several rounds, issue order alternating
            order = (0, 1) if rep % 2 == 0 else (1, 0)
            for i in order:
                d, t = dev[i]
                cwl.cwl_apply(d["X"], d["W"], d["A"], d["B"], t, window, Y=Y[i], workspace=ws[i], status_word=status[i],
                              stream=streams[i])
        torch.cuda.synchronize()
    assert [int(s.item()) for s in status] == [0, 0]
    for i, (h, t) in enumerate(probs):
        T = h["X"].shape[0]
        rows = np.unique(np.concatenate([[0, T - 1], np.random.default_rng(i).integers(0, T, 24),
                                         t["offsets"][1:-1], t["offsets"][1:-1] + 3])).astype(np.int32)
        ref = oracle.apply(h["X"], h["W"], h["A"], h["B"], host_table(t), window, rows=rows)
        check_output(y_to_f64(Y[i][torch.from_numpy(rows.astype(np.int64)).cuda()]), ref, label=f"two streams, call {i}")
