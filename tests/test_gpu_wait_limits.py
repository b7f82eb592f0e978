"""What the kernels do after a bounded wait ran out, exercised without losing anything.

``dq_debug_set_wait_limits(limit, 1)`` declares the FIRST wait of every consumer (a warp or a CTA)
lost without a look at its barrier, while the copy it waited for is valid and lands a moment
later.  The kernel must then raise DQ_STAT_WAIT, decide to leave in all threads that would
otherwise meet at a barrier, wait (with the ordinary limit) for every copy it has issued, and
return: the call completes, nothing outside the output buffers is touched, and the very next
call with the normal limits gives the right answer on the same context.  No copy is made to
fail and nothing hangs: the ordinary limit here is 50 ms, far more than any copy needs.
"""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

SEED = 0x7157_11_0A17
SEGS = [70, 4097, 31, 12345, 3 * 4096 + 77, 1 << 18]
LIMIT_NS = 50_000_000


@pytest.fixture(scope="module")
def G(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    import gpu_util
    return gpu_util


@pytest.fixture()
def short_first_wait(G):
    G.dq.debug_set_wait_limits(LIMIT_NS, True)
    yield
    G.dq.debug_set_wait_limits()          # back to the defaults, whatever the test did


def _grads(ref, M, seed):
    rng = np.random.default_rng(seed)
    g = np.zeros((M, ref.D32), np.float32)
    for o, n in zip(ref.offsets, SEGS):
        g[:, o: o + n] = rng.standard_normal((M, n)).astype(np.float32)
    return g


def _expect_wait_status_then_recover(G, r, call, check):
    """`call` under the short first wait raises DQ_STAT_WAIT (if any first wait was lost) and
    returns; the same call afterwards, with normal limits, passes `check`."""
    torch.cuda.synchronize()
    r.clear_status()
    call()
    torch.cuda.synchronize()                       # the kernel returned: nothing hangs
    st = r.read_status()
    assert st & ~G.dq.STAT_WAIT == 0, "only the wait bit may be raised, got %d" % st
    assert r.guards_intact()
    G.dq.debug_set_wait_limits()
    r.clear_status()
    check(call())
    assert r.read_status() == 0 and r.guards_intact()
    return st


@pytest.mark.parametrize("bucket", [512, 4096])
def test_bucket_norms_after_a_lost_first_wait(G, short_first_wait, bucket):
    ref = oracle.Layout(SEGS, bucket)
    g = _grads(ref, 3, bucket)
    want = oracle.bucket_norms(ref, g)
    r = G.GpuRound(SEGS, bucket, 3)
    r.set_grads(g)
    st = _expect_wait_status_then_recover(
        G, r, r.norms, lambda got: np.testing.assert_allclose(got, want, rtol=1e-6))
    assert st & G.dq.STAT_WAIT            # the copies of a cold start never land within one look


@pytest.mark.parametrize("bucket", [512, 2048, 4096])
def test_quantizers_after_a_lost_first_wait(G, short_first_wait, bucket):
    ref = oracle.Layout(SEGS, bucket)
    M, b = 2, 5
    g = _grads(ref, M, 10 + bucket)
    norms = oracle.bucket_norms(ref, g)
    want = oracle.quantize_pack(ref, g, norms, b, SEED, 1)
    nw = ref.packed_words(b)
    r = G.GpuRound(SEGS, bucket, M)
    r.set_grads(g)
    r.set_norms(norms)
    r.set_b(b)
    st = _expect_wait_status_then_recover(
        G, r, lambda: r.quantize(SEED, 1), lambda got: np.testing.assert_array_equal(got[:, :nw], want))
    assert st & G.dq.STAT_WAIT
    # fused norms + quantizer (per-warp tiles, teams of two and of four warps)
    G.dq.debug_set_wait_limits(LIMIT_NS, True)

    def fused():
        got_norms, packed = r.norms_quantize(SEED, 1)
        return got_norms.copy(), packed.copy()

    def check(res):
        got_norms, packed = res
        np.testing.assert_allclose(got_norms, norms, rtol=1e-6)
        np.testing.assert_array_equal(packed[:, :nw], oracle.quantize_pack(ref, g, got_norms, b, SEED, 1))

    st = _expect_wait_status_then_recover(G, r, fused, check)
    assert st & G.dq.STAT_WAIT


@pytest.mark.parametrize("M,b", [(3, 4), (16, 2), (5, 16)])
def test_average_and_update_after_a_lost_first_wait(G, short_first_wait, M, b):
    bucket = 512
    ref = oracle.Layout(SEGS, bucket)
    g = _grads(ref, M, 100 + M)
    norms = oracle.bucket_norms(ref, g)
    packed = oracle.quantize_pack(ref, g, norms, b, SEED, 2)
    want = oracle.unpack_dequant_average(ref, packed, norms, b)
    r = G.GpuRound(SEGS, bucket, M)
    full = np.zeros((M, r.pstride), np.uint32)
    full[:, : packed.shape[1]] = packed
    r.set_packed(full)
    r.set_norms(norms)
    r.set_b(b)
    st = _expect_wait_status_then_recover(
        G, r, lambda: r.average(fill=0.0).copy(), lambda got: _assert_rel_l2(G, got, want))
    assert st & G.dq.STAT_WAIT
    # the update epilogue waits for the tile of x as well
    G.dq.debug_set_wait_limits(LIMIT_NS, True)
    x = np.linspace(-1.0, 1.0, ref.D32, dtype=np.float32)
    lr = 0.25
    want_x = oracle.unpack_average_update(ref, packed, norms, b, lr, x)
    st = _expect_wait_status_then_recover(
        G, r, lambda: r.update(lr, x).copy(),
        lambda got: np.testing.assert_allclose(got, want_x, rtol=0, atol=1e-6 * lr * float(np.abs(want).max()) + 1.2e-7 * 2.0))
    assert st & G.dq.STAT_WAIT


def _assert_rel_l2(G, got, want):
    assert G.rel_l2(got, want) <= 1e-6


def test_limits_are_restored(G):
    """With the defaults back in place a whole round runs clean (guards against a leaked setting)."""
    G.dq.debug_set_wait_limits()
    ref = oracle.Layout(SEGS, 512)
    g = _grads(ref, 2, 5)
    r = G.GpuRound(SEGS, 512, 2)
    r.set_grads(g)
    r.set_b(4)
    norms, packed = r.norms_quantize(SEED, 0)
    r.average()
    assert r.read_status() == 0 and r.guards_intact()
