"""GPU parity at full workload sizes, in the launch configuration the benchmark times.

The small cases of ``test_gpu_parity.py`` cover every code path element by element; the
cases here show that nothing changes when the grids are full, the tile ranges long and
the indices large:
  * the benchmark workload (ResNet-18 shape, M = 8, bucket 512) through ``Round.step_fused``
    (one pass norms+quantize+pack, average, bit rule on a second stream), every output
    compared with the oracle, which finishes this size in seconds;
  * the VGG-16 and text-classifier shapes (M = 16, buckets 2048 and 1024) the same way;
  * the bandwidth-sweep sizes that the oracle cannot hold in host memory (d = 2^30 at M = 1,
    d = 2^26 at M = 32): the oracle checks a prefix of every worker word for word (codes
    depend only on an element's own bucket, worker, index and the step, so a prefix of the
    layout is a smaller problem with the same answer), and properties that hold for every
    element are checked over the whole array on the device: |Q(v) - v| <= norm/s,
    padding of the staging buffers untouched, mean error within 5 sigma of zero.
Tolerances are those stated in ``test_gpu_parity.py``.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2107_14575_b200 import dq, workloads as W
from paper_2107_14575_b200.pipeline import Round

pytestmark = pytest.mark.gpu

NORM_RTOL = 1e-6
AVG_RTOL = 1e-6
SEED = 0x0DDB_A11_5EED


@pytest.fixture(scope="module", autouse=True)
def _lib(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")


def _calibrated_rule(w, norms, t, x0=6.0):
    G2 = float((norms.astype(np.float64) ** 2).sum() / w.M)
    eps_hat = w.T * w.alpha ** (w.T - 1) * G2 / x0 ** 2
    return eps_hat, dq.Rule.dynamic(w.T, t, eps_hat, w.alpha)


def _full_round(w, b0, steps=2):
    """``steps`` rounds of Round.step_fused on workload ``w``; every output of every round against the oracle."""
    ref = oracle.Layout(w.segments, w.bucket)
    rnd = Round(w.segments, w.bucket, w.M)
    rnd.packed.fill_(-1)
    rnd.bits_(dq.Rule.fixed(b0))
    b = b0
    eps_hat = None
    for t in range(steps):
        g = W.make_grads(w, ref.offsets, ref.D32, step=t, pad_value=float("nan"))
        gd = torch.from_numpy(g).cuda()
        want_norms = oracle.bucket_norms(ref, g)
        if eps_hat is None:
            eps_hat, _ = _calibrated_rule(w, want_norms, 0)
        rule_next = dq.Rule.dynamic(w.T, t + 1, eps_hat, w.alpha)
        out = rnd.step_fused(gd, rule_next, SEED, t).cpu().numpy()
        torch.cuda.synchronize()
        assert rnd.read_status() == 0
        norms = rnd.norms.cpu().numpy()
        packed = rnd.packed.cpu().numpy().view(np.uint32)
        nw = ref.packed_words(b)

        np.testing.assert_allclose(norms, want_norms, rtol=NORM_RTOL, atol=0)
        # words: bit-exact against the oracle driven with the norms the kernel wrote
        want_packed = oracle.quantize_pack(ref, g, norms, b, SEED, t)
        assert np.array_equal(packed[:, :nw], want_packed)
        if t == 0:
            assert np.all(packed[:, nw:] == 0xFFFFFFFF)      # nothing written past the words in use
        # average
        want_out = oracle.unpack_dequant_average(ref, want_packed, norms, b)
        err = np.linalg.norm(out.astype(np.float64) - want_out) / max(np.linalg.norm(want_out), 1e-300)
        assert err <= AVG_RTOL, err
        # and element by element (a single element off by a level would not move the L2 ratio at
        # this size): within 1e-6 of the largest of its bucket's M norms -- the scale of the fp32 sums
        # behind it -- plus the rounding of the result itself
        scale = np.zeros(ref.D32)
        top = norms.max(axis=0).astype(np.float64)
        for k in range(ref.nb):
            s0, n = int(ref.bucket_start[k]), int(ref.bucket_len[k])
            scale[s0: s0 + n] = top[k]
        bound = 1e-6 * scale + 2.0 ** -23 * np.abs(want_out) + 1e-300
        worst = np.abs(out.astype(np.float64) - want_out) - bound
        assert np.all(worst <= 0), (int(np.argmax(worst)), float(worst.max()))
        # next b: the rule on the same norms
        b_next, s_next, _ = oracle.choose_bits(norms, w.T, t + 1, eps_hat, w.alpha)
        assert rnd.bits() == b_next
        b = b_next
    return b


def test_bench_workload_full_size_two_rounds():
    w = W.config_resnet18()
    assert w.M == 8 and w.bucket == 512 and sum(w.segments) == 11173962
    _full_round(w, b0=4, steps=2)


@pytest.mark.parametrize("b0", [7, 16])
def test_bench_workload_full_size_other_widths(b0):
    _full_round(W.config_resnet18(), b0=b0, steps=1)


def test_vgg16_full_size():
    w = W.config_vgg16()
    assert w.M == 16 and w.bucket == 2048
    _full_round(w, b0=4, steps=1)


def test_text_classifier_full_size():
    w = W.config_text()
    assert w.M == 16 and w.bucket == 1024
    _full_round(w, b0=5, steps=1)


def _device_normal(M, d, seed):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    g = torch.empty((M, d), dtype=torch.float32, device="cuda")
    for m in range(M):
        g[m].normal_(0.0, 1.0, generator=gen)
    return g


@pytest.mark.parametrize("d,M,bucket,b,prefix", [
    (1 << 30, 1, 512, 4, 1 << 22),
    (1 << 30, 1, 4096, 16, 1 << 22),
    (1 << 28, 1, 128, 1, 1 << 22),
    (1 << 28, 1, 4096, 6, 1 << 22),
    (1 << 26, 32, 512, 3, 1 << 20),
    (1 << 26, 32, 128, 8, 1 << 20),
    (1 << 26, 32, 4096, 4, 1 << 20),          # teams of four warps per bucket
    (1 << 26, 32, 2048, 5, 1 << 20),          # teams of two
])
def test_sweep_sizes_prefix_parity_and_whole_array_properties(d, M, bucket, b, prefix):
    s = (1 << (b - 1)) - 1
    rnd = Round([d], bucket, M, max_bits=b)
    L = rnd.layout
    g = _device_normal(M, d, seed=d % 1000 + M)
    rnd.packed.fill_(-1)
    rnd.bits_(dq.Rule.fixed(b))
    rnd.norms_quantize_(g, SEED, 3)
    torch.cuda.synchronize()
    assert rnd.read_status() == 0

    # ---- prefix of every worker, word for word
    ref = oracle.Layout([prefix], bucket)
    gp = g[:, :prefix].cpu().numpy()
    want_norms = oracle.bucket_norms(ref, gp)
    norms_p = rnd.norms[:, : ref.nb].cpu().numpy()
    np.testing.assert_allclose(norms_p, want_norms, rtol=NORM_RTOL, atol=0)
    want_packed = oracle.quantize_pack(ref, gp, norms_p, b, SEED, 3)
    got = rnd.packed[:, : ref.packed_words(b)].cpu().numpy().view(np.uint32)
    assert np.array_equal(got, want_packed)
    # ---- worker 0 over its whole length, word for word (every boundary between the ranges of the warps
    #      and CTAs that share it, and its end), where the oracle takes a few seconds
    if d <= (1 << 28):
        ref0 = oracle.Layout([d], bucket)
        g0 = g[:1].cpu().numpy()
        norms0 = rnd.norms[:1].cpu().numpy()
        np.testing.assert_allclose(norms0, oracle.bucket_norms(ref0, g0), rtol=NORM_RTOL, atol=0)
        want0 = oracle.quantize_pack(ref0, g0, norms0, b, SEED, 3)
        got0 = rnd.packed[:1, : ref0.packed_words(b)].cpu().numpy().view(np.uint32)
        assert np.array_equal(got0, want0)
        if M == 1 and b > 1:
            # one worker: the whole average against the oracle, element by element (bound as in _full_round)
            rnd.average_()
            torch.cuda.synchronize()
            assert rnd.read_status() == 0
            want_avg = oracle.unpack_dequant_average(ref0, want0, norms0, b)
            got_avg = rnd.out[:d].cpu().numpy().astype(np.float64)
            bound = 1e-6 * np.repeat(norms0[0].astype(np.float64), bucket)[:d] + 2.0 ** -23 * np.abs(want_avg) + 1e-300
            assert np.all(np.abs(got_avg - want_avg[:d]) <= bound)
            del want_avg, got_avg, bound
        del g0, want0, got0

    # nothing written past the words in use
    nw = L.packed_words(b)
    if rnd.packed_stride > nw:
        assert bool((rnd.packed[:, nw:] == -1).all())

    # ---- the separate norms kernel gives the same norms at this size
    fused_norms = rnd.norms.clone()
    rnd.norms_(g)
    assert torch.equal(rnd.norms, fused_norms)
    # ---- and the separate quantizer, given those norms, the same words
    fused_packed = rnd.packed[:, :nw].clone()
    rnd.packed.fill_(-1)
    rnd.quantize_(g, SEED, 3)
    torch.cuda.synchronize()
    assert rnd.read_status() == 0
    assert torch.equal(rnd.packed[:, :nw], fused_packed)
    del fused_packed

    # ---- whole array, M > 1: the average of the workers' Q(v) lies within the mean of their levels of the
    #      mean gradient (every Q(v) within one level of its v), and is unbiased
    if M > 1 and b > 1:
        rnd.average_()
        torch.cuda.synchronize()
        assert rnd.read_status() == 0
        q = rnd.out[:d]
        mean_g = g.mean(dim=0)
        step = (rnd.norms / s).mean(dim=0).repeat_interleave(bucket)[:d]
        diff = q - mean_g
        # (fp32 roundings of positions, products and of the two means: 4 ulp of s levels and 1e-5 absolute cover them)
        assert bool((diff.abs() <= step * (1.0 + 4.0 * s * 2.0 ** -23) + 1e-5).all())
        mean_err = float((diff / step).double().mean())
        assert abs(mean_err) <= 5 * 0.5 / np.sqrt(float(M) * d) + 1e-6
        del mean_g, step, diff

    # ---- whole array, M = 1 only (the average of one worker is Q(v) itself)
    if M == 1:
        rnd.average_()
        torch.cuda.synchronize()
        assert rnd.read_status() == 0
        q = rnd.out[:d]
        if b == 1:
            assert bool((q == 0).all())
            return
        step = (rnd.norms[0] / s).repeat_interleave(bucket)[:d]          # one level of each element's bucket
        err = (q - g[0]).abs()
        # one level, plus the fp32 rounding of position and product (|x| <= s, so 4 ulp of s levels covers it)
        assert bool((err <= step * (1.0 + 4.0 * s * 2.0 ** -23)).all())
        # unbiased: the mean error in units of a level is within 5 sigma of 0 (sigma <= 1/2 per element)
        mean_err = float(((q - g[0]) / step).double().mean())
        assert abs(mean_err) <= 5 * 0.5 / np.sqrt(d)
        # the average's prefix against the oracle as well
        want_out = oracle.unpack_dequant_average(ref, want_packed, norms_p, b)
        got_out = rnd.out[:prefix].cpu().numpy()
        rel = np.linalg.norm(got_out - want_out) / np.linalg.norm(want_out)
        assert rel <= AVG_RTOL


def test_bench_workload_full_size_with_parameter_update():
    """Round.step_fused with the update of Eq. 2 in the server step, full bench workload."""
    w = W.config_resnet18()
    ref = oracle.Layout(w.segments, w.bucket)
    rnd = Round(w.segments, w.bucket, w.M)
    b, lr = 5, 0.1
    rnd.bits_(dq.Rule.fixed(b))
    g = W.make_grads(w, ref.offsets, ref.D32, step=0)
    x = np.random.default_rng(1).normal(size=ref.D32).astype(np.float32) * 1e-2
    xd = torch.from_numpy(x).cuda()
    got = rnd.step_fused(torch.from_numpy(g).cuda(), dq.Rule.fixed(b), SEED, 0, params=xd, lr=lr)
    torch.cuda.synchronize()
    assert rnd.read_status() == 0 and got is xd
    norms = rnd.norms.cpu().numpy()
    packed = rnd.packed.cpu().numpy().view(np.uint32)[:, : ref.packed_words(b)]
    assert np.array_equal(packed, oracle.quantize_pack(ref, g, norms, b, SEED, 0))
    want = oracle.unpack_average_update(ref, packed, norms, b, lr, x)
    avg = oracle.unpack_dequant_average(ref, packed, norms, b)
    tol = 1e-6 * lr * np.abs(avg).max() + 2.0 ** -23 * np.abs(want) + 1e-30
    assert np.all(np.abs(got.cpu().numpy().astype(np.float64) - want) <= tol)


def test_bench_step_at_its_full_size_every_word_and_every_element():
    """The bench's own workload and call -- d = 2^26, M = 32, bucket 512, b = 4, one step_fused -- against the
    oracle over everything it writes: 4.2 M norms, 2^28 packed words bit for bit, 2^26 averaged elements each
    within its bound, and the next bit width.  (About 20 GB of host memory and half a minute of the oracle.)"""
    import psutil
    if psutil.virtual_memory().available < (48 << 30):
        pytest.skip("needs 48 GB of free host memory")
    d, M, bucket, b = 1 << 26, 32, 512, 4
    rnd = Round([d], bucket, M, max_bits=b)
    g = _device_normal(M, d, seed=77)
    rnd.packed.fill_(-1)
    rnd.bits_(dq.Rule.fixed(b))
    T, t_next = 100, 1
    rnd.norms_(g)
    G2 = float((rnd.norms.double() ** 2).sum().item() / M)
    eps_hat = T * G2 / 6.5 ** 2                    # x = 6.5: half a level below s(4) = 7, so the rule stays at b = 4
    out = rnd.step_fused(g, dq.Rule.dynamic(T, t_next, eps_hat, 1.0), SEED, 0)
    torch.cuda.synchronize()
    assert rnd.read_status() == 0

    ref = oracle.Layout([d], bucket)
    gh = g.cpu().numpy()
    del g
    norms = rnd.norms.cpu().numpy()
    np.testing.assert_allclose(norms, oracle.bucket_norms(ref, gh), rtol=NORM_RTOL, atol=0)
    want_packed = oracle.quantize_pack(ref, gh, norms, b, SEED, 0)
    del gh
    nw = ref.packed_words(b)
    got_packed = rnd.packed[:, :nw].cpu().numpy().view(np.uint32)
    assert np.array_equal(got_packed, want_packed)
    del got_packed
    if rnd.packed_stride > nw:
        assert bool((rnd.packed[:, nw:] == -1).all())
    want_out = oracle.unpack_dequant_average(ref, want_packed, norms, b)
    del want_packed
    got_out = out[:d].cpu().numpy().astype(np.float64)
    rel = np.linalg.norm(got_out - want_out[:d]) / np.linalg.norm(want_out[:d])
    assert rel <= AVG_RTOL
    bound = 1e-6 * np.repeat(norms.max(axis=0).astype(np.float64), bucket)[:d] + 2.0 ** -23 * np.abs(want_out[:d]) + 1e-300
    assert np.all(np.abs(got_out - want_out[:d]) <= bound)
    b_next, _, _ = oracle.choose_bits(norms, T, t_next, eps_hat, 1.0)
    assert rnd.bits() == b_next == b
