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


def test_a_round_can_be_captured_in_a_cuda_graph(dqlib):
    """The calls of a round allocate nothing and never synchronise, so a stream capture takes them
    (the bit rule on its side stream included); a replay writes what the eager calls wrote."""
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2107_14575_b200.pipeline import Round
    dq = dqlib
    w = W.scaled_down(W.config_resnet18(M=3), 16)
    rnd = Round(w.segments, w.bucket, w.M)
    D32 = rnd.layout.D32
    g = torch.randn((w.M, D32), generator=torch.Generator().manual_seed(9)).mul_(0.02).cuda()
    T, alpha = 50, 0.93
    rnd.norms_(g)
    G2 = float((rnd.norms.double() ** 2).sum().item() / w.M)
    rule = dq.Rule.dynamic(T, 30, T * alpha ** (T - 1) * G2 / 36.0, alpha)
    rnd.bits_(dq.Rule.fixed(4))
    cur0 = rnd._cur
    want = rnd.step_fused(g, rule, 3, 12).clone()          # eager; also creates the side stream and its events
    want_packed, want_norms, want_b = rnd.packed.clone(), rnd.norms.clone(), rnd._b.clone()
    torch.cuda.synchronize()

    rnd._cur = cur0                                        # same (b, s) slot as the eager round read
    rnd._b[cur0].copy_(torch.tensor([4, 7, 0, 0], dtype=torch.int32))
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=st):
        rnd.step_fused(g, rule, 3, 12)
    rnd.out.zero_(); rnd.packed.zero_(); rnd.norms.zero_()
    torch.cuda.synchronize()
    graph.replay()
    torch.cuda.synchronize()
    nw = rnd.layout.packed_words(4)                        # words beyond the stream are never written
    assert torch.equal(rnd.out, want) and torch.equal(rnd.norms, want_norms)
    assert torch.equal(rnd.packed[:, :nw], want_packed[:, :nw])
    assert torch.equal(rnd._b[1 - cur0], want_b[1 - cur0])  # the next b came out of the captured bit rule
    assert rnd.read_status() == 0
