"""The host-buffer entry of the pipeline (``Round.step_host``): uploads, rounds and downloads of
successive calls overlap on their own streams, and every call must still return exactly what the
same round on device-resident gradients returns."""
import numpy as np
import pytest
import torch

from paper_2107_14575_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_step_host_overlaps_calls_without_mixing_them(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2107_14575_b200.pipeline import Round
    dq = dqlib
    w = W.scaled_down(W.config_resnet18(M=4), 16)
    a = Round(w.segments, w.bucket, w.M)
    b = Round(w.segments, w.bucket, w.M)
    D32 = a.layout.D32
    gen = torch.Generator().manual_seed(5)
    steps = 7
    host = [torch.randn((w.M, D32), generator=gen).mul_(0.01 * (i + 1)).pin_memory() for i in range(steps)]
    rule = dq.Rule.fixed(5)
    a.bits_(rule)
    b.bits_(rule)
    outs = []
    for i in range(steps):                               # queued back to back, no synchronisation in between
        outs.append((i, a.step_host(host[i], rule, 77, i)))
    a.sync_host()
    # the last two results are still in their buffers; the earlier ones were overwritten by design
    want = {}
    for i in range(steps):
        want[i] = b.step_fused(host[i].cuda(), rule, 77, i).clone()
    torch.cuda.synchronize()
    for i, t in outs[-2:]:
        assert torch.equal(t, want[i].cpu())
    assert outs[-1][1].data_ptr() != outs[-2][1].data_ptr() and outs[-1][1].data_ptr() == outs[-3][1].data_ptr()
    # reading every result as it becomes valid: synchronise after each call
    c = Round(w.segments, w.bucket, w.M)
    c.bits_(rule)
    for i in range(steps):
        t = c.step_host(host[i], rule, 77, i)
        c.sync_host()
        assert torch.equal(t, want[i].cpu())
    assert a.read_status() == 0 and c.read_status() == 0
