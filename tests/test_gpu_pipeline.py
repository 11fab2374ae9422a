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
