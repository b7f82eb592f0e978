"""GPU parity: the CUDA library against the CPU oracle, through the C ABI.

Acceptance (stated once, used throughout):
  * packed words are bit-exact when the quantizer is driven with the oracle's norms;
  * bucket norms agree to 1e-6 relative;
  * with the GPU's own norms a code may differ by one only where x + v lies within
    1e-6 + |x| * delta + 2 ulp(x) of an integer, x = sgn*s|g|/norm the position on the
    level grid (an fp32 product), v the uniform draw and delta the relative difference
    of the two norms of that bucket (<= 1e-6): the window by which x itself moves;
  * the bit width b is identical when the rule is driven with the oracle's norms;
  * the averaged gradient agrees to 1e-6 relative L2.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2107_14575_b200 import workloads as W

pytestmark = pytest.mark.gpu

NORM_RTOL = 1e-6
AVG_RTOL = 1e-6
SEED = 0x1234_5678_9ABC_DEF0


@pytest.fixture(scope="module")
def G(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    import gpu_util
    return gpu_util


def _make(w, bucket=None, pad_value=0.0, step=0, stride_extra=0):
    ref = oracle.Layout(w.segments, bucket or w.bucket)
    stride = ref.D32 + stride_extra
    g = W.make_grads(w, ref.offsets, ref.D32, step=step, pad_value=pad_value, row_stride=stride)
    return ref, g


RAGGED = [70, 32, 1, 100, 4097, 31, 0, 64, 1000, 5, 12345]


def _cases():
    yield "flat-small", W.config_flat(d=1000, M=2, bucket=64, sigma=1.0)
    yield "flat-one-element", W.config_flat(d=1, M=1, bucket=32, sigma=1.0)
    yield "flat-31", W.config_flat(d=31, M=3, bucket=32, sigma=1.0)
    yield "flat-33", W.config_flat(d=33, M=3, bucket=32, sigma=1.0)
    yield "flat-tiles", W.config_flat(d=70001, M=3, bucket=512, sigma=0.1)       # several CTAs and a ragged tail
    yield "flat-b4096", W.config_flat(d=3 * 4096 + 77, M=2, bucket=4096, sigma=0.1)
    rag = W.config_flat(d=1, M=4, bucket=96, sigma=0.3)
    rag.segments = RAGGED
    yield "ragged-b96", rag
    yield "resnet/64", W.scaled_down(W.config_resnet18(M=3), 64)
    yield "vgg/256", W.scaled_down(W.config_vgg16(M=5), 256)
    yield "text/128", W.scaled_down(W.config_text(M=2), 128)


CASES = dict(_cases())


# ------------------------------------------------------------------- norms

@pytest.mark.parametrize("name", sorted(CASES))
def test_norms(G, name):
    w = CASES[name]
    ref, g = _make(w, pad_value=3e30, stride_extra=64)          # padding must be ignored
    r = G.GpuRound(w.segments, w.bucket, w.M, stride=ref.D32 + 64)
    r.set_grads(g)
    got = r.norms()
    want = oracle.bucket_norms(ref, g)
    assert np.all(np.abs(got - want) <= NORM_RTOL * want)
    assert r.read_status() == 0 and r.guards_intact()
    got2 = r.norms()
    assert np.array_equal(got, got2)                              # deterministic


@pytest.mark.parametrize("bucket", [32, 64, 96, 128, 160, 512, 1024, 4096])
def test_norms_bucket_sizes(G, bucket):
    w = W.config_flat(d=3 * 4096 + 1234, M=2, bucket=bucket, sigma=2.0)
    ref, g = _make(w)
    r = G.GpuRound(w.segments, bucket, w.M)
    r.set_grads(g)
    got, want = r.norms(), oracle.bucket_norms(ref, g)
    assert np.all(np.abs(got - want) <= NORM_RTOL * want)


def test_norms_nonfinite_sets_status(G):
    w = W.config_flat(d=4096, M=1, bucket=512)
    ref, g = _make(w)
    g[0, 700] = np.inf
    r = G.GpuRound(w.segments, w.bucket, 1)
    r.set_grads(g)
    got = r.norms()
    assert np.isinf(got[0, 1]) and np.isfinite(np.delete(got[0], 1)).all()
    assert r.read_status() & G.dq.STAT_NONFINITE


# ---------------------------------------------------- quantize + pack, exact

@pytest.mark.parametrize("b", list(range(1, 17)))
@pytest.mark.parametrize("name", ["flat-small", "flat-33", "flat-tiles", "ragged-b96", "resnet/64"])
def test_quantize_pack_bit_exact_with_oracle_norms(G, name, b):
    w = CASES[name]
    ref, g = _make(w, pad_value=-7.5)
    norms = oracle.bucket_norms(ref, g)
    want = oracle.quantize_pack(ref, g, norms, b, SEED, 3)
    r = G.GpuRound(w.segments, w.bucket, w.M)
    r.set_grads(g)
    r.set_norms(norms)
    r.set_b(b)
    got = r.quantize(SEED, 3, fill=-1)
    nw = ref.packed_words(b)
    assert np.array_equal(got[:, :nw], want[:, :nw])
    assert np.all(got[:, nw:] == 0xFFFFFFFF)                      # words beyond b*D32/32 untouched
    assert r.read_status() == 0 and r.guards_intact()


@pytest.mark.parametrize("name", sorted(CASES))
def test_quantize_pack_bit_exact_all_cases_b5(G, name):
    w = CASES[name]
    ref, g = _make(w)
    norms = oracle.bucket_norms(ref, g)
    r = G.GpuRound(w.segments, w.bucket, w.M)
    r.set_grads(g)
    r.set_norms(norms)
    for b, step in ((5, 0), (2, 1), (11, 0xFFFFFFFF)):
        r.set_b(b)
        got = r.quantize(SEED + b, step)
        want = oracle.quantize_pack(ref, g, norms, b, SEED + b, step)
        nw = ref.packed_words(b)
        assert np.array_equal(got[:, :nw], want[:, :nw])
    assert r.guards_intact()


def test_config1_round_trip(G):
    """d = 2^20, M = 4, N(0, 0.01), bucket 512, fixed b in {2, 4, 8}: one full round."""
    w = W.config_flat()
    ref, g = _make(w)
    r = G.GpuRound(w.segments, w.bucket, w.M)
    r.set_grads(g)
    norms_gpu = r.norms()
    norms = oracle.bucket_norms(ref, g)
    assert np.all(np.abs(norms_gpu - norms) <= NORM_RTOL * norms)
    for b in w.fixed_b:
        assert r.bits(G.dq.Rule.fixed(b)) == (b, (1 << (b - 1)) - 1)
        # exact leg: oracle norms
        r.set_norms(norms)
        got = r.quantize(0, 0)
        want = oracle.quantize_pack(ref, g, norms, b, 0, 0)
        nw = ref.packed_words(b)
        assert np.array_equal(got[:, :nw], want[:, :nw])
        out = r.average()
        assert G.rel_l2(out, oracle.unpack_dequant_average(ref, want, norms, b)) <= AVG_RTOL
        # the quantized average approximates the true mean within the Lemma 1 bound (4 sigma)
        err2 = float(((out.astype(np.float64) - g.mean(0)) ** 2).sum())
        s = (1 << (b - 1)) - 1
        bound = (w.bucket / (4.0 * s * s)) * float((norms.astype(np.float64) ** 2).sum()) / w.M ** 2
        assert err2 <= bound * 1.05


# --------------------------------------- quantize with the GPU's own norms

@pytest.mark.parametrize("name,b", [("flat-tiles", 4), ("resnet/64", 6), ("vgg/256", 3), ("text/128", 9),
                                     ("ragged-b96", 16)])
def test_quantize_with_gpu_norms_differs_only_at_ties(G, name, b):
    w = CASES[name]
    ref, g = _make(w)
    r = G.GpuRound(w.segments, w.bucket, w.M)
    r.set_grads(g)
    norms_gpu = r.norms().copy()
    norms = oracle.bucket_norms(ref, g)
    assert np.all(np.abs(norms_gpu - norms) <= NORM_RTOL * norms)
    r.set_b(b)
    got = r.quantize(SEED, 9)
    codes_ref, x, v = oracle.quantize(ref, g, norms, b, SEED, 9, want_x_v=True)
    for m in range(w.M):
        codes = oracle.unpack(got[m], ref.D32, b)
        diff = np.nonzero(codes != codes_ref[m])[0]
        if diff.size:
            dl = codes[diff].astype(np.int64) - codes_ref[m][diff].astype(np.int64)
            assert np.all(np.abs(dl) == 1)
            # a relative norm difference delta moves x = sgn*s|g|/norm by |x|*delta, so
            # floor(x + v) can change only where x + v lies within |x|*delta (+ the fp32
            # spacing of x) of an integer; for small |x| this is the plain 1e-6 window
            k = np.searchsorted(ref.bucket_start, diff, side="right") - 1
            delta = np.abs(norms_gpu[m][k].astype(np.float64) - norms[m][k]) / norms[m][k]
            z = x[m][diff].astype(np.float64) + v[m][diff].astype(np.float64)
            margin = np.abs(z - np.round(z))
            ulp = np.spacing(np.abs(x[m][diff])).astype(np.float64)     # x itself is an fp32 product
            widening = 1.001 * np.abs(x[m][diff]) * delta + 2 * ulp
            assert np.all(margin < 1e-6 + widening)
            # where that widening is itself below 1e-6 (small |x|, i.e. small b) the contract's literal
            # window |frac - u| < 1e-6 (doubled for the two sources) must hold as stated
            literal = widening < 1e-6
            assert np.all(margin[literal] < 2e-6)
        assert diff.size <= 1e-4 * ref.D32 + 2
    # and driven with its own norms the GPU reproduces the oracle driven with those same norms
    want = oracle.quantize_pack(ref, g, norms_gpu, b, SEED, 9)
    assert np.array_equal(got[:, : ref.packed_words(b)], want)


# ------------------------------------------- norms + quantize in one pass

@pytest.mark.parametrize("name", sorted(CASES))
def test_fused_norms_quantize_equals_the_two_passes(G, name):
    """dq_norms_quantize_pack writes the norms of dq_bucket_norms and the words of
    dq_quantize_pack for those norms, bit for bit; and the words are the oracle's for them."""
    w = CASES[name]
    ref, g = _make(w, pad_value=7e29)
    r = G.GpuRound(w.segments, w.bucket, w.M)
    r.set_grads(g)
    norms_sep = r.norms().copy()
    for b, step in ((4, 0), (1, 2), (7, 3), (16, 9)):
        r.set_b(b)
        packed_sep = r.quantize(SEED, step, fill=-1).copy()
        r.g_norms.view.fill_(-1.0)
        norms_fused, packed_fused = r.norms_quantize(SEED, step, fill=-1)
        assert np.array_equal(norms_fused, norms_sep)
        assert np.array_equal(packed_fused, packed_sep)
        nw = ref.packed_words(b)
        want = oracle.quantize_pack(ref, g, norms_fused, b, SEED, step)
        assert np.array_equal(packed_fused[:, :nw], want)
        assert np.all(packed_fused[:, nw:] == 0xFFFFFFFF)
    assert np.all(np.abs(norms_sep - oracle.bucket_norms(ref, g)) <= NORM_RTOL * oracle.bucket_norms(ref, g))
    assert r.read_status() == 0 and r.guards_intact()


@pytest.mark.parametrize("bucket", [32, 64, 128, 256, 1024, 2048, 4096, 96, 160])
def test_fused_bucket_sizes(G, bucket):
    w = W.config_flat(d=3 * 4096 + 1234, M=3, bucket=bucket, sigma=2.0)
    ref, g = _make(w)
    r = G.GpuRound(w.segments, bucket, w.M)
    r.set_grads(g)
    for b in (3, 8):
        r.set_b(b)
        norms, packed = r.norms_quantize(5, 1, fill=-1)
        ref_norms = oracle.bucket_norms(ref, g)
        assert np.all(np.abs(norms - ref_norms) <= NORM_RTOL * ref_norms)
        want = oracle.quantize_pack(ref, g, norms, b, 5, 1)
        assert np.array_equal(packed[:, : ref.packed_words(b)], want)
    assert r.read_status() == 0 and r.guards_intact()


def test_fused_step_order_of_algorithm_1(G):
    """quantize with b_t (one pass) -> average -> b_{t+1} from this step's norms."""
    w = CASES["resnet/64"]
    T = 10
    alpha = (2.4e-3) ** (1.0 / T)
    r = G.GpuRound(w.segments, w.bucket, w.M)
    b = 4                                                      # b_0, an input of Algorithm 1
    r.set_b(b)
    eps_hat = None
    for t in range(T):
        ref, g = _make(w, step=t)
        r.set_grads(g)
        norms, packed = r.norms_quantize(SEED, t)
        want = oracle.quantize_pack(ref, g, norms, b, SEED, t)
        assert np.array_equal(packed[:, : ref.packed_words(b)], want)
        out = r.average()
        assert G.rel_l2(out, oracle.unpack_dequant_average(ref, want, norms, b)) <= AVG_RTOL
        if eps_hat is None:
            G2 = float((norms.astype(np.float64) ** 2).sum() / w.M)
            eps_hat = T * alpha ** (T - 1) * G2 / 36.0
        if t + 1 < T:
            b_next = r.bits(G.dq.Rule.dynamic(T, t + 1, eps_hat, alpha))
            assert b_next[0] == oracle.choose_bits(norms, T, t + 1, eps_hat, alpha)[0]
            b = b_next[0]
    assert b > 4 and r.read_status() == 0 and r.guards_intact()


# ------------------------------------------------------------------ bit rule

def test_choose_bits_matches_oracle(G):
    w = CASES["resnet/64"]
    ref, g = _make(w)
    norms = oracle.bucket_norms(ref, g)
    r = G.GpuRound(w.segments, w.bucket, w.M)
    r.set_norms(norms)
    G2 = float((norms.astype(np.float64) ** 2).sum() / w.M)
    T, alpha = 100, (2.4e-3) ** (1 / 100)
    eps_hat = T * alpha ** (T - 1) * G2 / 36.0                     # x(t = 0) = 6 -> b = 4
    seen = set()
    for t in list(range(0, T, 7)) + [T - 1]:
        want = oracle.choose_bits(norms, T, t, eps_hat, alpha)
        got = r.bits(G.dq.Rule.dynamic(T, t, eps_hat, alpha))
        assert got == want[:2], (t, got, want)
        seen.add(got[0])
    assert min(seen) == 4 and max(seen) >= 8
    # clamps, fixed b, scale extremes
    for kw in (dict(b_min=5, b_max=6), dict(b_min=2, b_max=3), dict(b_min=16, b_max=16)):
        for t in (0, T - 1):
            assert r.bits(G.dq.Rule.dynamic(T, t, eps_hat, alpha, **kw)) == \
                oracle.choose_bits(norms, T, t, eps_hat, alpha, **kw)[:2]
    for eps in (1e-30, 1e30):
        assert r.bits(G.dq.Rule.dynamic(T, 0, eps, alpha)) == oracle.choose_bits(norms, T, 0, eps, alpha)[:2]
    for fb in (1, 7, 16):
        assert r.bits(G.dq.Rule.fixed(fb)) == (fb, (1 << (fb - 1)) - 1)
    assert r.read_status() == 0 and r.guards_intact()


def test_choose_bits_many_norms_and_zero(G):
    # more than one reduction chunk; all-zero norms clamp to b_min
    w = W.config_flat(d=32 * 70000, M=3, bucket=32, sigma=1.0)
    ref, g = _make(w)
    norms = oracle.bucket_norms(ref, g)
    r = G.GpuRound(w.segments, w.bucket, w.M)
    r.set_norms(norms)
    for t, eps in ((0, 10.0), (5, 1e3), (9, 1e5)):
        assert r.bits(G.dq.Rule.dynamic(10, t, eps, 0.8)) == oracle.choose_bits(norms, 10, t, eps, 0.8)[:2]
    r.set_norms(np.zeros_like(norms))
    assert r.bits(G.dq.Rule.dynamic(10, 3, 1.0, 0.8)) == (2, 1)
    n2 = norms.copy()
    n2[1, 5] = np.nan
    r.set_norms(n2)
    assert r.bits(G.dq.Rule.dynamic(10, 3, 1.0, 0.8)) == (16, 32767)
    assert r.read_status() & G.dq.STAT_NONFINITE


@pytest.mark.parametrize("b", [2, 5, 9, 16])
def test_scale_division_is_exact_over_the_norm_range(G, b):
    """inv = RZ(s / norm) decides every code; one bucket of 32 elements per norm, norms over the whole
    exponent range, quotients that are exact, and the bounds of the kernel's inline division."""
    s = (1 << (b - 1)) - 1
    nbk = 1 << 15
    rng = np.random.default_rng(b)
    mant = (1.0 + rng.random(nbk)).astype(np.float32)
    expo = rng.integers(-95, 120, size=nbk)
    norms = np.ldexp(mant, expo).astype(np.float32)
    special = []
    for k in (-60, -7, 0, 3, 40):
        special += [np.ldexp(1.0, k), np.ldexp(float(s), k)]                 # quotient a power of two
        special += [np.ldexp(float(s) / m, k) for m in (1, 3, 7, 31, 151) if s % m == 0]   # exact quotients
        special += [np.ldexp(3.0, k), np.ldexp(1.0 - 2.0 ** -24, k), np.ldexp(1.0 + 2.0 ** -23, k)]
    special += [2.0 ** -100, np.nextafter(np.float32(2.0 ** -100), np.float32(0)), 2.0 ** -120, 0.0,
                2.0 ** 125, np.nextafter(np.float32(2.0 ** 125), np.float32(np.inf)), 2.0 ** 126, 3.0e38]
    norms[: len(special)] = np.array(special, np.float32)
    u = rng.random((nbk, 32)).astype(np.float32)
    u[:, 0] = 1.0                                                              # an entry as large as the norm
    u[:, 1] = np.float32(1.0 - 2.0 ** -24)
    sign = np.where(rng.random((nbk, 32)) < 0.5, -1.0, 1.0).astype(np.float32)
    g = (norms[:, None] * u * sign).astype(np.float32).reshape(1, -1)
    assert np.all(np.abs(g.reshape(nbk, 32)) <= norms[:, None])
    ref = oracle.Layout([nbk * 32], 32)
    r = G.GpuRound([nbk * 32], 32, 1)
    r.set_grads(g)
    r.set_norms(norms.reshape(1, -1))
    r.set_b(b)
    got = r.quantize(SEED, 7, fill=0)
    want = oracle.quantize_pack(ref, g, norms.reshape(1, -1), b, SEED, 7)
    assert np.array_equal(got[:, : ref.packed_words(b)], want)
    assert r.read_status() == 0 and r.guards_intact()


# ------------------------------------------------- unpack + dequantize + average

@pytest.mark.parametrize("b", list(range(1, 17)))
@pytest.mark.parametrize("M", [1, 4, 32])
def test_average_matches_oracle(G, M, b):
    w = W.config_flat(d=9000 + 13, M=M, bucket=128, sigma=0.5, seed=M)
    ref, g = _make(w)
    norms = oracle.bucket_norms(ref, g)
    packed = oracle.quantize_pack(ref, g, norms, b, SEED, 1)
    r = G.GpuRound(w.segments, w.bucket, M, packed_stride=(ref.packed_words(b) + 3) // 4 * 4 + 8)
    full = np.full((M, r.pstride), 0xA5A5A5A5, np.uint32)
    full[:, : ref.packed_words(b)] = packed
    r.set_packed(full)
    r.set_norms(norms)
    r.set_b(b)
    out = r.average(fill=123.0)
    want = oracle.unpack_dequant_average(ref, packed, norms, b)
    assert G.rel_l2(out, want) <= AVG_RTOL
    assert np.all(out[9013:] == 0)                                 # padding is +0
    if b == 1:
        assert np.all(out == 0)
    assert r.read_status() == 0 and r.guards_intact()


@pytest.mark.parametrize("name,M,b", [("ragged-b96", 4, 3), ("resnet/64", 8, 5), ("vgg/256", 16, 7),
                                       ("text/128", 16, 4), ("flat-b4096", 2, 12)])
def test_average_multi_tensor(G, name, M, b):
    w = CASES[name]
    w = W.Workload(**{**w.__dict__})
    w.M = M
    ref, g = _make(w)
    norms = oracle.bucket_norms(ref, g)
    packed = oracle.quantize_pack(ref, g, norms, b, 77, 0)
    r = G.GpuRound(w.segments, w.bucket, M)
    full = np.zeros((M, r.pstride), np.uint32)
    full[:, : ref.packed_words(b)] = packed
    r.set_packed(full)
    r.set_norms(norms)
    r.set_b(b)
    out = r.average()
    want = oracle.unpack_dequant_average(ref, packed, norms, b)
    assert G.rel_l2(out, want) <= AVG_RTOL
    assert np.array_equal(out, r.average())                        # deterministic


def test_on_level_workers_average_exactly(G):
    # identical workers whose entries sit on quantization levels come back exactly
    b, s = 4, 7
    row = np.zeros((1, 64), np.float32)
    row[0, :3] = [2 * 0.25, -3 * 0.25, 6 * 0.25]
    row[0, 32:35] = [-6.0, 2.0, 3.0]
    g = np.ascontiguousarray(np.broadcast_to(row, (8, 64)))
    r = G.GpuRound([64], 32, 8)
    r.set_grads(g)
    r.norms()
    r.set_b(b)
    r.quantize(5, 5)
    assert np.array_equal(r.average(), row[0])


# ------------------------------------------- average + parameter update (Eq. 2)

def _update_tolerance(lr, avg, want):
    # the fp32 average is within 1e-6 of the fp64 one (relative to the bucket's scale, bounded here by
    # the largest entry), and the result is rounded to fp32 once on each side
    return 1e-6 * abs(lr) * np.abs(avg).max() + 2.0 ** -23 * np.abs(want) + 1e-30


@pytest.mark.parametrize("b", [1, 2, 3, 4, 5, 8, 11, 16])
@pytest.mark.parametrize("M", [1, 4, 32])
def test_average_update_matches_oracle(G, M, b):
    w = W.config_flat(d=9000 + 13, M=M, bucket=128, sigma=0.5, seed=M)
    ref, g = _make(w)
    norms = oracle.bucket_norms(ref, g)
    packed = oracle.quantize_pack(ref, g, norms, b, SEED, 1)
    r = G.GpuRound(w.segments, w.bucket, M, packed_stride=(ref.packed_words(b) + 3) // 4 * 4 + 8)
    full = np.full((M, r.pstride), 0xA5A5A5A5, np.uint32)
    full[:, : ref.packed_words(b)] = packed
    r.set_packed(full)
    r.set_norms(norms)
    r.set_b(b)
    rng = np.random.default_rng(b * 100 + M)
    x = rng.normal(size=ref.D32).astype(np.float32)
    x[9013:] = 123.0                                               # padding of the parameters
    lr = 0.37
    got = r.update(lr, x)
    want = oracle.unpack_average_update(ref, packed, norms, b, lr, x)
    avg = oracle.unpack_dequant_average(ref, packed, norms, b)
    assert np.all(np.abs(got.astype(np.float64) - want) <= _update_tolerance(lr, avg, want))
    assert np.array_equal(got[9013:], x[9013:])                    # padding keeps its value
    if b == 1:
        assert np.array_equal(got, x)
    else:
        assert not np.array_equal(got[:9013], x[:9013])
    assert r.read_status() == 0 and r.guards_intact()


@pytest.mark.parametrize("name,M,b", [("ragged-b96", 4, 3), ("resnet/64", 8, 5), ("vgg/256", 16, 7),
                                       ("text/128", 16, 4), ("flat-b4096", 2, 12)])
def test_average_update_multi_tensor(G, name, M, b):
    w = CASES[name]
    w = W.Workload(**{**w.__dict__})
    w.M = M
    ref, g = _make(w)
    norms = oracle.bucket_norms(ref, g)
    packed = oracle.quantize_pack(ref, g, norms, b, 77, 0)
    r = G.GpuRound(w.segments, w.bucket, M)
    full = np.zeros((M, r.pstride), np.uint32)
    full[:, : ref.packed_words(b)] = packed
    r.set_packed(full)
    r.set_norms(norms)
    r.set_b(b)
    x = np.random.default_rng(5).normal(size=ref.D32).astype(np.float32) * 0.01
    lr = -0.05                                                     # ascent is allowed: eta is just a number
    got = r.update(lr, x)
    want = oracle.unpack_average_update(ref, packed, norms, b, lr, x)
    avg = oracle.unpack_dequant_average(ref, packed, norms, b)
    assert np.all(np.abs(got.astype(np.float64) - want) <= _update_tolerance(lr, avg, want))
    # the same average as the plain call: x - lr * out, rounded once
    out = r.average()
    assert np.array_equal(got, (x.astype(np.float64) - np.float64(np.float32(lr)) * out).astype(np.float32))
    assert r.read_status() == 0 and r.guards_intact()


def test_update_on_level_workers_is_exact_and_rejects_bad_eta(G):
    b = 4
    row = np.zeros((1, 64), np.float32)
    row[0, :3] = [2 * 0.25, -3 * 0.25, 6 * 0.25]
    row[0, 32:35] = [-6.0, 2.0, 3.0]
    g = np.ascontiguousarray(np.broadcast_to(row, (8, 64)))
    r = G.GpuRound([64], 32, 8)
    r.set_grads(g)
    r.norms()
    r.set_b(b)
    r.quantize(5, 5)
    x = np.arange(64, dtype=np.float32) * 0.125 - 3.0
    assert np.array_equal(r.update(0.5, x), x - np.float32(0.5) * row[0])
    from paper_2107_14575_b200 import dq
    for bad in (float("nan"), float("inf")):
        with pytest.raises(dq.DQError) as e:
            r.update(bad, x)
        assert e.value.code == dq.ERR_RANGE


# ------------------------------------------------------- whole step, device b

@pytest.mark.parametrize("name", ["resnet/64", "vgg/256", "text/128"])
def test_dynamic_step_matches_oracle_pipeline(G, name):
    """norms -> rule -> quantize -> average with b living on the device only."""
    w = CASES[name]
    T = 12
    alpha = (2.4e-3) ** (1.0 / T)
    r = G.GpuRound(w.segments, w.bucket, w.M)
    eps_hat = None
    bs = []
    for t in range(T):
        ref, g = _make(w, step=t)
        r.set_grads(g)
        norms_gpu = r.norms().copy()
        norms = oracle.bucket_norms(ref, g)
        assert np.all(np.abs(norms_gpu - norms) <= NORM_RTOL * norms)
        if eps_hat is None:
            G2 = float((norms.astype(np.float64) ** 2).sum() / w.M)
            eps_hat = T * alpha ** (T - 1) * G2 / 36.0
        b, s = r.bits(G.dq.Rule.dynamic(T, t, eps_hat, alpha))
        want_b, want_s, x = oracle.choose_bits(norms_gpu, T, t, eps_hat, alpha)
        assert (b, s) == (want_b, want_s)
        bs.append(b)
        got = r.quantize(SEED, t)
        want = oracle.quantize_pack(ref, g, norms_gpu, b, SEED, t)
        assert np.array_equal(got[:, : ref.packed_words(b)], want)
        out = r.average()
        assert G.rel_l2(out, oracle.unpack_dequant_average(ref, want, norms_gpu, b)) <= AVG_RTOL
    assert bs[0] == 4 and bs[-1] > bs[0]
    assert r.read_status() == 0 and r.guards_intact()


# ----------------------------------------------------------- device conditions

def test_bad_bits_and_capacity_write_nothing(G):
    w = CASES["flat-small"]
    ref, g = _make(w)
    r = G.GpuRound(w.segments, w.bucket, w.M, packed_stride=ref.packed_words(4))
    r.set_grads(g)
    r.norms()
    for bad in (0, 17, -3):
        r.clear_status()
        r.set_b(bad)
        got = r.quantize(1, 1, fill=-1)
        out = r.average(fill=9.0)
        assert np.all(got == 0xFFFFFFFF) and np.all(out == 9.0)
        assert r.read_status() == G.dq.STAT_BAD_BITS
    r.clear_status()
    r.set_b(5)                                                      # needs 5*D32/32 words, 4*D32/32 given
    got = r.quantize(1, 1, fill=-1)
    out = r.average(fill=9.0)
    assert np.all(got == 0xFFFFFFFF) and np.all(out == 9.0)
    assert r.read_status() == G.dq.STAT_CAPACITY
    r.clear_status()
    r.set_b(4)
    r.quantize(1, 1)
    r.average()
    assert r.read_status() == 0 and r.guards_intact()


def test_zero_stride_workers_and_streams(G):
    # stride 0: every worker reads the same buffer but draws from its own stream
    w = W.config_flat(d=4096, M=1, bucket=256, sigma=1.0)
    ref, g = _make(w)
    M = 6
    r = G.GpuRound(w.segments, w.bucket, M, stride=0)
    r.grads = torch.from_numpy(g).cuda()
    r.stride = 0
    norms = r.norms()
    assert np.all(norms == norms[0])
    r.set_b(3)
    got = r.quantize(3, 0)
    gb = np.ascontiguousarray(np.broadcast_to(g, (M, ref.D32)))
    want = oracle.quantize_pack(ref, gb, norms, 3, 3, 0)
    assert np.array_equal(got[:, : ref.packed_words(3)], want)
    assert not np.array_equal(got[0], got[1])
    # a side stream gives the same words
    st = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        got2 = r.quantize(3, 0)
    st.synchronize()
    assert np.array_equal(got, got2)
