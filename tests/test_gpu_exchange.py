"""The sharded path (one worker per rank) on one GPU: the ranks of ``exchange.ShardedRound`` run
turn by turn in this process over a loopback transport, so no kernel ever waits for another.
What it must reproduce, bit for bit: the unsharded path over the same workers (same words,
same norms, same averaged gradient, same next b), and through it the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2107_14575_b200 import workloads as W

pytestmark = pytest.mark.gpu

SEED = 0x51AB_0000_7777_0001
RAGGED = [70, 32, 1, 100, 4097, 31, 0, 64, 1000, 5, 12345]


@pytest.fixture(scope="module")
def G(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    import gpu_util
    return gpu_util


def _grads(segs, M, ref, seed, scale=0.05):
    rng = np.random.default_rng(seed)
    g = np.zeros((M, ref.D32), np.float32)
    for o, n in zip(ref.offsets, segs):
        g[:, o: o + n] = (rng.standard_normal((M, n)) * scale).astype(np.float32)
    return g


@pytest.mark.parametrize("first", [0, 1, 5, 4095])
def test_first_worker_selects_the_oracles_stream(G, first):
    """Worker m of a call with first_worker = f draws what worker f + m draws in the oracle."""
    segs, bucket, b = RAGGED, 64, 5
    ref = oracle.Layout(segs, bucket)
    M = 2
    g_all = _grads(segs, first + M, ref, 1)
    norms_all = oracle.bucket_norms(ref, g_all)
    want = oracle.quantize_pack(ref, g_all, norms_all, b, SEED, 3)[first: first + M] if first < 64 else None
    if want is None:                                   # a far-away worker index: only two oracle rows are needed
        g_two = g_all[first: first + M]
        # the oracle numbers workers from 0: give it rows [first, first + M) in place by padding with views
        big = np.zeros((first + M, ref.D32), np.float32)
        big[first:] = g_two
        nb = oracle.bucket_norms(ref, big)
        want = oracle.quantize_pack(ref, big, nb, b, SEED, 3)[first:]
        norms_all = nb
    r = G.GpuRound(segs, bucket, M)
    r.set_grads(np.ascontiguousarray(g_all[first: first + M]))
    r.set_norms(norms_all[first: first + M])
    r.set_b(b)
    nw = ref.packed_words(b)
    G.dq.quantize_pack_worker(r.lay, r.grads, r.stride, M, r.g_norms.view, r.g_b.view, SEED, 3, first,
                              r.g_packed.view, r.pstride, r.status)
    got = r.g_packed.view.cpu().numpy().view(np.uint32).reshape(M, r.pstride)[:, :nw]
    assert np.array_equal(got, want)
    G.dq.norms_quantize_pack_worker(r.lay, r.grads, r.stride, M, r.g_b.view, SEED, 3, first, r.g_norms.view,
                                    r.g_packed.view, r.pstride, r.status)
    got = r.g_packed.view.cpu().numpy().view(np.uint32).reshape(M, r.pstride)[:, :nw]
    if first + M <= 64:
        # with the GPU's own norms the words are those of the unsharded call's rows
        full = G.GpuRound(segs, bucket, first + M)
        full.set_grads(g_all)
        full.set_b(b)
        _, packed_full = full.norms_quantize(SEED, 3)
        assert np.array_equal(got, packed_full[first:, :nw])
    assert r.read_status() == 0 and r.guards_intact()


CASES = [
    ("ragged-b64-w3", RAGGED, 64, 3, "l2"),
    ("ragged-b4096-w2", RAGGED, 4096, 2, "l2"),
    ("flat-w4", [3 * 4096 + 77], 512, 4, "l2"),
    ("few-buckets-w8", [100], 32, 8, "l2"),                  # some ranks get no range at all
    ("ragged-linf-w3", RAGGED, 96, 3, "linf"),
    ("ragged-whole-w2", RAGGED, 0, 2, "l2"),
]


@pytest.mark.parametrize("name,segs,bucket,world,p", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("b", [2, 5, 12])
def test_sharded_round_equals_the_unsharded_one(G, name, segs, bucket, world, p, b):
    from paper_2107_14575_b200 import exchange
    from paper_2107_14575_b200.pipeline import Round
    dq = G.dq
    norm = dq.NORM_L2 if p == "l2" else dq.NORM_LINF
    ref = oracle.Layout(segs, oracle.whole_tensor_bucket(segs) if bucket == 0 else bucket)
    g = _grads(segs, world, ref, 10 * world + b)
    dev_g = torch.from_numpy(g).cuda()

    # the unsharded path: all workers in one call
    one = Round(segs, bucket, world, norm=norm)
    one.bits_(dq.Rule.fixed(b))
    one.norms_quantize_(dev_g, SEED, 7)
    one.average_()
    T, t, alpha = 40, 10, 0.9
    G2 = float((one.norms.double() ** 2).sum().item() / world)
    eps_hat = T * alpha ** (T - 1) * G2 / 25.0 if G2 > 0 else 1.0
    rule = dq.Rule.dynamic(T, t, eps_hat, alpha)

    # the sharded path: one ShardedRound per rank, stepped turn by turn
    hub = exchange.LoopbackTransport(world)
    ranks = [exchange.ShardedRound(segs, bucket, hub.bind(r), r, world, norm=norm) for r in range(world)]
    for r in ranks:
        r.set_bits(b)
    for i, r in enumerate(ranks):
        r.quantize_(dev_g[i], SEED, 7)
    for r in ranks:
        r.share_norms_()
    for r in ranks:
        r.exchange_(b)
    for r in ranks:
        r.average_()
    for r in ranks:
        r.gather_()
    for r in ranks:
        r.assemble_()
    torch.cuda.synchronize()
    nw = ref.packed_words(b)
    want_packed = one.packed.cpu().numpy().view(np.uint32)
    want_out = one.out.cpu().numpy()
    for i, r in enumerate(ranks):
        assert r.read_status() == 0
        assert np.array_equal(r.packed_local.cpu().numpy().view(np.uint32)[:nw], want_packed[i, :nw])
        assert torch.equal(r.norms_all, one.norms)
        assert np.array_equal(r.out.cpu().numpy(), want_out)          # bit for bit, on every rank
    # the next b is the same everywhere and equals the unsharded rule's
    one.bits_(rule)
    for r in ranks:
        r.bits_(rule)
        assert r.read_bits() == one.bits()
    # and the whole thing is the oracle's average
    kind = oracle.NORM_L2 if p == "l2" else oracle.NORM_LINF
    norms = one.norms.cpu().numpy()
    want = oracle.unpack_dequant_average(ref, oracle.quantize_pack(ref, g, norms, b, SEED, 7), norms, b)
    assert G.rel_l2(want_out, want) <= 1e-6 or not np.any(want)
    assert np.all(np.abs(norms - oracle.bucket_norms(ref, g, kind)) <= 1e-6 * np.abs(norms))


def test_sharded_step_on_a_model_shape(G):
    """``step`` end to end over three ranks on the ResNet-18 shape (scaled down), dynamic b."""
    from paper_2107_14575_b200 import exchange
    dq = G.dq
    w = W.scaled_down(W.config_resnet18(M=3), 32)
    ref = oracle.Layout(w.segments, w.bucket)
    g = W.make_grads(w, ref.offsets, ref.D32)
    dev_g = torch.from_numpy(g).cuda()
    world, b = 3, 4
    hub = exchange.LoopbackTransport(world)
    ranks = [exchange.ShardedRound(w.segments, w.bucket, hub.bind(r), r, world) for r in range(world)]
    norms = oracle.bucket_norms(ref, g)
    T, alpha = 100, (2.4e-3) ** 0.01
    eps_hat = T * alpha ** (T - 1) * float((norms.astype(np.float64) ** 2).sum() / world) / 36.0
    rule = dq.Rule.dynamic(T, 60, eps_hat, alpha)
    for r in ranks:
        r.set_bits(b)
    # the phases of step(), rank after rank (a collective completes when the last rank has called it)
    for i, r in enumerate(ranks):
        r.quantize_(dev_g[i], SEED, 0)
    for phase in ("share_norms_", "average_", "gather_", "assemble_"):
        if phase == "average_":
            for r in ranks:
                r.exchange_(b)
        for r in ranks:
            getattr(r, phase)()
    for r in ranks:
        r.bits_(rule)
    torch.cuda.synchronize()
    gpu_norms = ranks[0].norms_all.cpu().numpy()
    want = oracle.unpack_dequant_average(ref, oracle.quantize_pack(ref, g, gpu_norms, b, SEED, 0), gpu_norms, b)
    bo, _, _ = oracle.choose_bits(gpu_norms, T, 60, eps_hat, alpha)
    for r in ranks:
        assert r.read_status() == 0
        assert G.rel_l2(r.out.cpu().numpy(), want) <= 1e-6
        assert r.read_bits() == bo


@pytest.mark.parametrize("b", [3, 8])
def test_sharded_step_over_nccl_with_one_rank(G, b):
    """The NCCL transport itself (not the loopback): a process group of one rank on this GPU drives
    ``ShardedRound.step`` through ``DistTransport`` -- all-gather of the norms, all-to-all of the packed
    range into this rank's own memory, average, all-gather of the result -- and must reproduce the
    unsharded round bit for bit and, through it, the oracle."""
    import os
    import socket

    import torch.distributed as dist
    from paper_2107_14575_b200 import exchange
    from paper_2107_14575_b200.pipeline import Round
    dq = G.dq
    if dist.is_initialized():
        pytest.skip("a process group is already up in this process")
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    os.environ.setdefault("NCCL_NVLS_ENABLE", "0")
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1,
                            device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        segs, bucket = RAGGED + [3 * 4096 + 77], 512
        ref = oracle.Layout(segs, bucket)
        g = _grads(segs, 1, ref, 40 + b)
        dev_g = torch.from_numpy(g).cuda()
        one = Round(segs, bucket, 1)
        one.bits_(dq.Rule.fixed(b))
        one.norms_quantize_(dev_g, SEED, 2)
        one.average_()
        T, alpha = 50, 0.93
        G2 = float((one.norms.double() ** 2).sum().item())
        eps_hat = T * alpha ** (T - 1) * G2 / 30.0
        rule = dq.Rule.dynamic(T, 20, eps_hat, alpha)

        r = exchange.ShardedRound(segs, bucket, exchange.DistTransport(), 0, 1)
        r.set_bits(b)
        assert r.dev_b[:2].tolist() == [b, (1 << (b - 1)) - 1]         # (b, s) written by the library
        out = r.step(dev_g[0], b, SEED, 2).clone()
        out2 = r.step(dev_g[0], b, SEED, 2, next_rule=rule).clone()      # a second round reuses the staging buffer
        torch.cuda.synchronize()
        assert r.read_status() == 0
        one.bits_(rule)
        assert r.read_bits() == one.bits()                               # the next b, from the gathered norms
        nw = ref.packed_words(b)
        assert np.array_equal(r.packed_local.cpu().numpy().view(np.uint32)[:nw],
                              one.packed.cpu().numpy().view(np.uint32)[0, :nw])
        assert torch.equal(r.norms_all, one.norms)
        assert torch.equal(out, one.out) and torch.equal(out2, one.out)
        norms = one.norms.cpu().numpy()
        want = oracle.unpack_dequant_average(ref, oracle.quantize_pack(ref, g, norms, b, SEED, 2), norms, b)
        assert G.rel_l2(out.cpu().numpy(), want) <= 1e-6
    finally:
        dist.destroy_process_group()
