"""GPU parity for the other members of the quantizer family of Eq. 5: l_inf bucket norms
(separate pass and fused with the quantizer) and one norm per tensor, against the CPU oracle
through the C ABI.

Acceptance: l_inf norms are exact (a maximum involves no rounding), so with them the packed
words of the GPU's own norms are bit-exact too; l_2 norms of whole tensors agree to 1e-6
relative; packed words are bit-exact when the quantizer is driven with the oracle's norms;
the averaged gradient agrees to 1e-6 relative L2.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2107_14575_b200 import workloads as W

pytestmark = pytest.mark.gpu

SEED = 0x0BAD_CAFE_1234_5678
RAGGED = [70, 32, 1, 100, 4097, 31, 0, 64, 1000, 5, 12345]


@pytest.fixture(scope="module")
def G(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    import gpu_util
    return gpu_util


def _grads(segs, M, ref, seed, pad_value=0.0, scale=1.0):
    rng = np.random.default_rng(seed)
    g = np.full((M, ref.D32), pad_value, np.float32)
    for o, n in zip(ref.offsets, segs):
        g[:, o: o + n] = (rng.standard_normal((M, n)) * scale).astype(np.float32)
    return g


# ------------------------------------------------------------ l_inf, bucketed

@pytest.mark.parametrize("bucket", [32, 64, 96, 128, 160, 512, 1024, 2048, 4096])
def test_linf_bucket_norms_are_exact(G, bucket):
    segs = RAGGED + [3 * 4096 + 77]
    ref = oracle.Layout(segs, bucket)
    g = _grads(segs, 3, ref, bucket, pad_value=7e30)             # padding must be ignored
    r = G.GpuRound(segs, bucket, 3, norm=G.dq.NORM_LINF)
    r.set_grads(g)
    got = r.norms()
    assert np.array_equal(got, oracle.bucket_norms(ref, g, oracle.NORM_LINF))
    assert r.read_status() == 0 and r.guards_intact()


def test_linf_nan_and_inf_reach_the_status_word(G):
    segs = [4096]
    ref = oracle.Layout(segs, 512)
    for bad, bucket in ((np.nan, 512), (np.inf, 512), (np.nan, 96)):
        g = _grads(segs, 1, oracle.Layout(segs, bucket), 1)
        g[0, 700] = bad
        r = G.GpuRound(segs, bucket, 1, norm=G.dq.NORM_LINF)
        r.set_grads(g)
        got = r.norms()
        k = 700 // bucket
        assert not np.isfinite(got[0, k]) and np.isfinite(np.delete(got[0], k)).all()
        assert r.read_status() & G.dq.STAT_NONFINITE


@pytest.mark.parametrize("b", [1, 2, 3, 4, 5, 8, 11, 16])
@pytest.mark.parametrize("bucket", [64, 96, 512, 2048, 4096])
def test_linf_fused_norms_and_words_bit_exact(G, bucket, b):
    """dq_norms_quantize_pack on an l_inf layout: per-warp tile pipelines (64, 512), the
    teams of two warps (2048), teams of four warps (4096) and the two-pass route of other bucket sizes (96)."""
    segs = RAGGED + [5 * 4096 + 33]
    ref = oracle.Layout(segs, bucket)
    g = _grads(segs, 2, ref, 10 * bucket + b, pad_value=-3.25, scale=0.02)
    want_norms = oracle.bucket_norms(ref, g, oracle.NORM_LINF)
    want = oracle.quantize_pack(ref, g, want_norms, b, SEED, 5)
    r = G.GpuRound(segs, bucket, 2, norm=G.dq.NORM_LINF)
    r.set_grads(g)
    r.set_b(b)
    norms, packed = r.norms_quantize(SEED, 5, fill=-1)
    nw = ref.packed_words(b)
    assert np.array_equal(norms, want_norms)
    assert np.array_equal(packed[:, :nw], want)
    assert np.all(packed[:, nw:] == 0xFFFFFFFF)                  # nothing beyond the stream is touched
    assert r.read_status() == 0 and r.guards_intact()
    # the separate passes give the same words
    r.norms()
    assert np.array_equal(r.quantize(SEED, 5)[:, :nw], want)
    # and the average of those words is the oracle's
    out = r.average(fill=1e30)
    ref_out = oracle.unpack_dequant_average(ref, want, want_norms, b)
    assert G.rel_l2(out, ref_out) <= 1e-6 or not np.any(ref_out)


def test_linf_full_round_on_a_model_shape(G):
    w = W.scaled_down(W.config_resnet18(M=4), 32)
    ref = oracle.Layout(w.segments, w.bucket)
    g = W.make_grads(w, ref.offsets, ref.D32)
    r = G.GpuRound(w.segments, w.bucket, w.M, norm=G.dq.NORM_LINF)
    r.set_grads(g)
    r.set_b(4)
    norms, packed = r.norms_quantize(SEED, 0)
    want_norms = oracle.bucket_norms(ref, g, oracle.NORM_LINF)
    assert np.array_equal(norms, want_norms)
    want = oracle.quantize_pack(ref, g, want_norms, 4, SEED, 0)
    assert np.array_equal(packed[:, : ref.packed_words(4)], want)
    out = r.average()
    assert G.rel_l2(out, oracle.unpack_dequant_average(ref, want, want_norms, 4)) <= 1e-6
    # the l_inf grid is finer than the l_2 one: the quantization error of the average is smaller
    r2 = G.GpuRound(w.segments, w.bucket, w.M)
    r2.set_grads(g)
    r2.set_b(4)
    r2.norms_quantize(SEED, 0)
    out2 = r2.average()
    mean = g.astype(np.float64).mean(axis=0)
    assert np.linalg.norm(out - mean) < np.linalg.norm(out2 - mean)


# ------------------------------------------------------- one norm per tensor

WHOLE = [RAGGED, [1], [31], [4096], [4097], [300000, 7, 1100000], [1 << 20]]


@pytest.mark.parametrize("p", ["l2", "linf"])
@pytest.mark.parametrize("segs", WHOLE, ids=[str(i) for i in range(len(WHOLE))])
def test_tensor_norms(G, segs, p):
    kind_o = oracle.NORM_L2 if p == "l2" else oracle.NORM_LINF
    kind_g = G.dq.NORM_L2 if p == "l2" else G.dq.NORM_LINF
    ref = oracle.Layout(segs, oracle.whole_tensor_bucket(segs))
    M = 3
    g = _grads(segs, M, ref, len(segs), pad_value=-9e30, scale=0.5)
    r = G.GpuRound(segs, G.dq.BUCKET_WHOLE_TENSOR, M, norm=kind_g)
    assert r.lay.nb == ref.nb
    r.set_grads(g)
    got = r.norms()
    want = oracle.bucket_norms(ref, g, kind_o)
    if p == "linf":
        assert np.array_equal(got, want)
    else:
        assert np.all(np.abs(got - want) <= 1e-6 * want)
        # the norm dominates every entry of its tensor (the quantizer relies on it)
        k = 0
        for o, n in zip(ref.offsets, segs):
            if n:
                assert np.all(np.abs(g[:, o: o + n]).max(axis=1) <= got[:, k])
                k += 1
    assert r.read_status() == 0 and r.guards_intact()
    assert np.array_equal(got, r.norms())                        # deterministic


@pytest.mark.parametrize("p", ["l2", "linf"])
@pytest.mark.parametrize("b", [2, 5, 8, 13])
def test_whole_tensor_round(G, p, b):
    """norms -> bit rule -> quantize -> average on a whole-tensor layout."""
    kind_o = oracle.NORM_L2 if p == "l2" else oracle.NORM_LINF
    kind_g = G.dq.NORM_L2 if p == "l2" else G.dq.NORM_LINF
    segs = [70, 0, 33000, 5, 4096 * 9 + 1]
    ref = oracle.Layout(segs, oracle.whole_tensor_bucket(segs))
    M = 4
    g = _grads(segs, M, ref, b, pad_value=2.5, scale=0.01)
    r = G.GpuRound(segs, G.dq.BUCKET_WHOLE_TENSOR, M, norm=kind_g)
    r.set_grads(g)
    want_norms = oracle.bucket_norms(ref, g, kind_o)
    # exact words with the oracle's norms
    r.set_norms(want_norms)
    assert r.bits(G.dq.Rule.fixed(b)) == (b, (1 << (b - 1)) - 1)
    want = oracle.quantize_pack(ref, g, want_norms, b, SEED, 9)
    nw = ref.packed_words(b)
    assert np.array_equal(r.quantize(SEED, 9, fill=-1)[:, :nw], want)
    out = r.average(fill=-1e30)
    assert G.rel_l2(out, oracle.unpack_dequant_average(ref, want, want_norms, b)) <= 1e-6
    # with the GPU's own norms: identical for l_inf; for l_2 every code within one of the oracle's
    got_norms = r.norms()
    packed = r.quantize(SEED, 9)[:, :nw]
    if p == "linf":
        assert np.array_equal(packed, want)
    else:
        for m in range(M):
            c_gpu = oracle.unpack(packed[m], ref.D32, b).astype(np.int64)
            c_ref = oracle.unpack(want[m], ref.D32, b).astype(np.int64)
            assert np.max(np.abs(c_gpu - c_ref)) <= 1
            assert np.mean(c_gpu != c_ref) < 1e-3
    # the dynamic rule on these norms agrees with the oracle's
    T, t, alpha = 50, 20, 0.95
    G2 = float((want_norms.astype(np.float64) ** 2).sum() / M)
    eps_hat = T * alpha ** (T - 1) * G2 / 30.0
    r.set_norms(want_norms)
    bo, so, _ = oracle.choose_bits(want_norms, T, t, eps_hat, alpha)
    assert r.bits(G.dq.Rule.dynamic(T, t, eps_hat, alpha)) == (bo, so)
    assert r.read_status() == 0 and r.guards_intact()


def test_pipeline_round_with_whole_tensor_linf(G):
    """The Round object strings the same calls together (two passes for a whole-tensor layout)."""
    from paper_2107_14575_b200.pipeline import Round
    segs = [5000, 129, 70000]
    ref = oracle.Layout(segs, oracle.whole_tensor_bucket(segs))
    g = _grads(segs, 2, ref, 4, scale=0.1)
    rnd = Round(segs, G.dq.BUCKET_WHOLE_TENSOR, 2, norm=G.dq.NORM_LINF)
    dev_g = torch.from_numpy(g).cuda()
    rnd.bits_(G.dq.Rule.fixed(6))
    out = rnd.step_fused(dev_g, G.dq.Rule.fixed(6), SEED, 1).cpu().numpy()
    torch.cuda.synchronize()
    assert rnd.read_status() == 0
    norms = oracle.bucket_norms(ref, g, oracle.NORM_LINF)
    assert np.array_equal(rnd.norms.cpu().numpy(), norms)
    want = oracle.quantize_pack(ref, g, norms, 6, SEED, 1)
    assert np.array_equal(rnd.packed.cpu().numpy().view(np.uint32)[:, : ref.packed_words(6)], want)
    assert G.rel_l2(out, oracle.unpack_dequant_average(ref, want, norms, 6)) <= 1e-6
