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
