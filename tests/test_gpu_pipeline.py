"""HostPipeline (uploads, kernels and downloads of neighbouring steps overlapped on three streams, two device
slots) must return exactly what the plain one-stream sequence copy - step - copy returns."""
import numpy as np
import pytest
import torch

from paper_2601_21109_b200 import workloads as wl
from paper_2601_21109_b200.runner import HostPipeline, HotPath

pytestmark = pytest.mark.gpu


def test_pipelined_steps_equal_the_serial_result():
    w = wl.config2(T=640, V=4096, projections=[("q", 256, 256), ("gate", 256, 512), ("up", 256, 512), ("down", 512, 256)])
    plain = HotPath(w)
    plain.score_step()
    ths = np.percentile(plain.score.cpu().numpy(), [25, 50, 75]).astype(np.float32).tolist()
    plain.set_thresholds(ths)
    plain.step()
    torch.cuda.synchronize()
    want = [p.Y.cpu() for p in plain.projs]
    pipe = HostPipeline(w)
    for s in pipe.slots:
        s.set_thresholds(ths)
    for y in pipe.host_Y[0] + pipe.host_Y[1]:
        y.fill_(float("nan"))
    a, b = pipe.run(5)                                   # both slots are used, the last step lands in slot 0
    torch.cuda.synchronize()
    assert a.elapsed_time(b) > 0
    for slot in pipe.slots:
        assert int(slot.status.item()) == 0
    for k in (0, 1):
        for got, ref in zip(pipe.host_Y[k], want):
            assert torch.equal(got.view(torch.int16), ref.view(torch.int16))
    assert pipe.h2d_bytes == 640 * (256 + 512) * 2 + 640 * 4096 * 4
    assert pipe.d2h_bytes == 640 * (256 + 512 + 512 + 256) * 2


def test_a_captured_step_replays_to_the_same_outputs():
    # the whole step (score, partition, six apply launches and their memsets) as one CUDA graph
    w = wl.config2(T=640, V=4096, projections=[("q", 256, 256), ("gate", 256, 512), ("up", 256, 512), ("down", 512, 256)])
    hp = HotPath(w)
    hp.score_step()
    hp.set_thresholds(np.percentile(hp.score.cpu().numpy(), [25, 50, 75]).astype(np.float32).tolist())
    hp.step()
    torch.cuda.synchronize()
    want = [p.Y.clone() for p in hp.projs]
    graph = hp.capture()
    for p in hp.projs:
        p.Y.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert int(hp.status.item()) == 0
    for p, ref in zip(hp.projs, want):
        assert torch.equal(p.Y.view(torch.int16), ref.view(torch.int16))


def test_pipelined_decode_through_the_scheduler():
    """Decode slots advance their own scheduler state: after n pipelined steps a slot's outputs equal those of a
    plain runner stepped as often as that slot was (slot 0: steps 0, 2, 4; slot 1: steps 1, 3)."""
    w = wl.config4(T=48)
    w.policy = wl.Policy.ladder([8, 16, 32, 64], 32.0, [0.25, 0.5, 0.75], min_len=4, window=2)
    w.score = np.random.default_rng(11).uniform(0, 1, w.T).astype(np.float32)
    pipe = HostPipeline(w, streaming=True)
    pipe.run(5)
    torch.cuda.synchronize()
    for k, n_steps in ((0, 3), (1, 2)):
        plain = HotPath(w, streaming=True)
        for _ in range(n_steps):
            plain.step()
        torch.cuda.synchronize()
        assert int(plain.status.item()) == 0 and int(pipe.slots[k].status.item()) == 0
        for got, p in zip(pipe.host_Y[k], plain.projs):
            assert torch.equal(got.view(torch.int16), p.Y.cpu().view(torch.int16))
    assert pipe.h2d_bytes == 48 * (4096 + 11008) * 2 + 48 * 4
