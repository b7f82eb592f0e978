"""GPU parity of the norm kernels over the whole magnitude range of fp32 gradients.

The l_2 norm of Eq. 5 is a sum of squares, and fp32 squares leave the normal range for entries
below about 2^-63 and above 2^+64.  The kernels reduce such buckets a second time with a
power-of-two scale; these tests drive the GPU's OWN norm kernels (every route: separate pass,
fused with the quantizer, plain-load kernels, one norm per tensor) on buckets whose entries sit
between 2^-99 and 2^-55 and between 2^+55 and 2^+99, mixed with ordinary buckets, and check

* norms within 1e-6 relative of the oracle's (fp64 accumulation),
* every norm at least as large as every entry of its bucket (the encoder relies on it),
* packed words bit for bit equal to the oracle's when the oracle is driven with those norms,
* the averaged gradient within 1e-6 relative L2.
"""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

SEED = 0x5EED_0F_7A11_CA5E
RAGGED = [70, 32, 1, 100, 4097, 31, 0, 64, 1000, 5, 12345, 1]


@pytest.fixture(scope="module")
def G(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    import gpu_util
    return gpu_util


def _bucket_max(ref, g):
    """Largest magnitude of every bucket, [M, nb] (exact)."""
    return oracle.bucket_norms(ref, g, oracle.NORM_LINF)


def _extreme_grads(segs, M, ref, seed, pad_value=0.0):
    """N(0,1) entries times 2^e with one exponent per bucket: a third of the buckets tiny
    (e in [-99, -55]), a third huge (e in [55, 99]), a third ordinary (e in [-8, 8]); some buckets
    keep a single non-zero entry, some are all zero."""
    rng = np.random.default_rng(seed)
    g = np.full((M, ref.D32), pad_value, np.float32)
    for m in range(M):
        for k in range(ref.nb):
            s, n = int(ref.bucket_start[k]), int(ref.bucket_len[k])
            kind = rng.integers(0, 3)
            e = (rng.integers(-99, -54), rng.integers(55, 100), rng.integers(-8, 9))[kind]
            v = np.ldexp(rng.standard_normal(n), int(e)).astype(np.float32)
            shape = rng.integers(0, 8)
            if shape == 0:                       # a single entry carries the bucket
                keep = rng.integers(0, n)
                one = v[keep] if v[keep] != 0 else np.float32(np.ldexp(1.0, int(e)))
                v[:] = 0
                v[keep] = one
            elif shape == 1:
                v[:] = 0
            g[m, s: s + n] = v
    return g


def _check_norms(ref, g, got, want):
    assert np.all(np.isfinite(got))
    assert np.all(np.abs(got.astype(np.float64) - want) <= 1e-6 * want.astype(np.float64))
    assert np.all(got >= _bucket_max(ref, g)), "a norm is smaller than an entry of its bucket"


BUCKETS = [32, 64, 96, 160, 512, 1024, 2048, 4096]


@pytest.mark.parametrize("bucket", BUCKETS)
def test_l2_norms_of_tiny_and_huge_buckets(G, bucket):
    """dq_bucket_norms: the bulk-copy kernel (32 * 2^k) and the plain-load kernels (96, 160)."""
    segs = RAGGED + [3 * 4096 + 77]
    ref = oracle.Layout(segs, bucket)
    g = _extreme_grads(segs, 3, ref, bucket, pad_value=7e30)
    r = G.GpuRound(segs, bucket, 3)
    r.set_grads(g)
    got = r.norms()
    _check_norms(ref, g, got, oracle.bucket_norms(ref, g))
    assert r.read_status() == 0 and r.guards_intact()
    assert np.array_equal(got, r.norms())                        # deterministic


@pytest.mark.parametrize("b", [2, 4, 7, 12, 16])
@pytest.mark.parametrize("bucket", BUCKETS)
def test_fused_and_separate_words_with_the_gpus_own_norms(G, bucket, b):
    """dq_norms_quantize_pack (per-warp tiles, teams of two and of four warps, two-pass route) and
    dq_bucket_norms + dq_quantize_pack on the same inputs: same norms, and words equal to the
    oracle's when it is given those norms."""
    segs = RAGGED + [5 * 4096 + 33]
    ref = oracle.Layout(segs, bucket)
    M = 2
    g = _extreme_grads(segs, M, ref, 100 * bucket + b, pad_value=-3.25)
    r = G.GpuRound(segs, bucket, M)
    r.set_grads(g)
    r.set_b(b)
    norms, packed = r.norms_quantize(SEED, 3, fill=-1)
    norms = norms.copy()
    packed = packed.copy()
    _check_norms(ref, g, norms, oracle.bucket_norms(ref, g))
    nw = ref.packed_words(b)
    want = oracle.quantize_pack(ref, g, norms, b, SEED, 3)
    assert np.array_equal(packed[:, :nw], want)
    assert np.all(packed[:, nw:] == 0xFFFFFFFF)
    assert r.read_status() == 0 and r.guards_intact()
    # the separate passes: identical norms, identical words
    assert np.array_equal(r.norms(), norms)
    assert np.array_equal(r.quantize(SEED, 3)[:, :nw], want)
    # and the average of those words
    out = r.average(fill=1e30)
    ref_out = oracle.unpack_dequant_average(ref, want, norms, b)
    assert np.all(np.isfinite(out))
    assert G.rel_l2(out, ref_out) <= 1e-6
    assert r.read_status() == 0 and r.guards_intact()


@pytest.mark.parametrize("e", [-99, -90, -75, -64, -63, -55, 55, 63, 64, 80, 99])
@pytest.mark.parametrize("bucket", [64, 512, 4096, 96])
def test_uniform_magnitude_and_single_entries(G, bucket, e):
    """All buckets at one magnitude 2^e (so every tile takes the same route), with single-element
    tensors among them: an entry alone in its bucket is its own norm."""
    segs = [1, bucket, 1, 2 * bucket + 1, 4096 * 2]
    ref = oracle.Layout(segs, bucket)
    rng = np.random.default_rng(1000 + e)
    g = np.zeros((2, ref.D32), np.float32)
    for o, n in zip(ref.offsets, segs):
        g[:, o: o + n] = np.ldexp(rng.standard_normal((2, n)), e).astype(np.float32)
    r = G.GpuRound(segs, bucket, 2)
    r.set_grads(g)
    r.set_b(8)
    norms, packed = r.norms_quantize(SEED, 0)
    norms = norms.copy()
    _check_norms(ref, g, norms, oracle.bucket_norms(ref, g))
    assert norms[0, 0] == abs(g[0, 0]) and norms[1, 2] == abs(g[1, ref.offsets[2]])
    want = oracle.quantize_pack(ref, g, norms, 8, SEED, 0)
    assert np.array_equal(packed[:, : ref.packed_words(8)], want)
    assert np.array_equal(r.norms(), norms)
    assert r.read_status() == 0 and r.guards_intact()


@pytest.mark.parametrize("bucket", [512, 2048, 4096, 160])
def test_a_norm_beyond_fp32_is_infinite_like_the_oracles(G, bucket):
    """Entries near the top of the fp32 range: the norm overflows to infinity in the oracle
    (fp64 result rounded to fp32) and on the GPU alike, and the status word says so; buckets
    that are merely huge stay finite."""
    segs = [4 * bucket]
    ref = oracle.Layout(segs, bucket)
    g = np.zeros((1, ref.D32), np.float32)
    g[0, :bucket] = np.float32(2.0 ** 126)                      # norm 2^126 * sqrt(bucket): infinite
    g[0, bucket: 2 * bucket] = np.float32(2.0 ** 110)           # finite
    g[0, 2 * bucket] = np.float32(3.0e38)                       # alone: finite, its own norm
    want = oracle.bucket_norms(ref, g)
    r = G.GpuRound(segs, bucket, 1)
    r.set_grads(g)
    got = r.norms()
    assert np.isinf(want[0, 0]) and np.isinf(got[0, 0])
    assert np.all(np.abs(got[0, 1:] - want[0, 1:]) <= 1e-6 * want[0, 1:])
    assert got[0, 2] == np.float32(3.0e38)
    assert r.read_status() & G.dq.STAT_NONFINITE


@pytest.mark.parametrize("p", ["l2", "linf"])
def test_linf_and_tensor_norms_over_the_range(G, p):
    kind_o = oracle.NORM_L2 if p == "l2" else oracle.NORM_LINF
    kind_g = G.dq.NORM_L2 if p == "l2" else G.dq.NORM_LINF
    # bucketed l_inf: exact whatever the magnitude
    segs = RAGGED + [3 * 4096 + 77]
    if p == "linf":
        for bucket in (64, 96, 512, 4096):
            ref = oracle.Layout(segs, bucket)
            g = _extreme_grads(segs, 2, ref, bucket)
            r = G.GpuRound(segs, bucket, 2, norm=kind_g)
            r.set_grads(g)
            assert np.array_equal(r.norms(), oracle.bucket_norms(ref, g, kind_o))
            assert r.read_status() == 0
    # one norm per tensor: every tensor at its own magnitude
    segs = [70, 1, 33000, 5, 4096 * 9 + 1, 4096, 300000]
    ref = oracle.Layout(segs, oracle.whole_tensor_bucket(segs))
    rng = np.random.default_rng(7)
    g = np.full((3, ref.D32), -9e30, np.float32)
    for i, (o, n) in enumerate(zip(ref.offsets, segs)):
        e = (-99, 99, -70, 64, -60, 0, 90)[i]
        g[:, o: o + n] = np.ldexp(rng.standard_normal((3, n)), e).astype(np.float32)
    r = G.GpuRound(segs, G.dq.BUCKET_WHOLE_TENSOR, 3, norm=kind_g)
    r.set_grads(g)
    got = r.norms()
    want = oracle.bucket_norms(ref, g, kind_o)
    if p == "linf":
        assert np.array_equal(got, want)
    else:
        assert np.all(np.abs(got.astype(np.float64) - want) <= 1e-6 * want.astype(np.float64))
        for k, (o, n) in enumerate(zip(ref.offsets, segs)):
            assert np.all(np.abs(g[:, o: o + n]).max(axis=1) <= got[:, k])
    assert r.read_status() == 0 and r.guards_intact()
