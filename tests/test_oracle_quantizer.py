"""Pins for the oracle's norms, stochastic quantizer and average (CPU only).

What fixes the expected values: numpy's norm, Lemma 1 of the paper
(unbiasedness, per-coordinate variance p_r(1-p_r)/s^2, trace bound
d*||g||^2/(4 s^2), 1/W scaling of the average's variance), inputs lying
exactly on quantization levels, and brute force over every rounding outcome.
"""
import itertools

import numpy as np
import pytest

import oracle
from paper_2107_14575_b200 import workloads as W


def _values(codes, norm, b):
    """Eq. 5 written out with numpy for one bucket: norm * sgn * level / s,
    with the code holding s + sgn * level."""
    s = (1 << (b - 1)) - 1
    return (codes.astype(np.float64) - s) * float(norm) / s


# ----------------------------------------------------------------- norms (P6)

def test_norms_match_numpy():
    w = W.scaled_down(W.config_resnet18(M=3), 64)
    lay = oracle.Layout(w.segments, 64)
    g = W.make_grads(w, lay.offsets, lay.D32, pad_value=1e30)   # pads must be ignored
    norms = oracle.bucket_norms(lay, g)
    for m in range(w.M):
        for k in (0, 1, lay.nb // 2, lay.nb - 1):
            st, ln = lay.bucket_start[k], lay.bucket_len[k]
            ref = np.linalg.norm(g[m, st: st + ln].astype(np.float64))
            assert abs(norms[m, k] - ref) <= 1e-7 * ref + 1e-45
    # sum of squared bucket norms = squared norm of the whole tensor list (p = 2)
    valid = np.concatenate([g[0, o: o + n] for o, n in zip(lay.offsets, w.segments)]).astype(np.float64)
    assert abs((norms[0].astype(np.float64) ** 2).sum() - (valid ** 2).sum()) < 1e-6 * (valid ** 2).sum()


# ------------------------------------------------------- on-level inputs (P2)

# integer vectors L with sum L_j^2 = s^2 for s = 2^(b-1) - 1
_ON_LEVEL = {
    2: [1, 0, 0],            # s = 1
    3: [1, 2, 2],            # s = 3
    4: [2, 3, 6],            # s = 7
    5: [9, 12, 0],           # s = 15 = 3*(3,4,5)
    6: [30, 6, 5],           # s = 31
    7: [18, 27, 54],         # s = 63 = 9*(2,3,6)
    8: [127, 0, 0],
    9: [153, 204, 0],        # s = 255 = 51*(3,4,5)
    12: [0, 2047, 0],
    16: [4681 * 2, 4681 * 3, 4681 * 6],   # s = 32767 = 7*4681
}


@pytest.mark.parametrize("b", sorted(_ON_LEVEL))
def test_on_level_inputs_are_reproduced_exactly(b):
    s = (1 << (b - 1)) - 1
    L = np.array(_ON_LEVEL[b], np.int64)
    assert int((L * L).sum()) == s * s
    for c in (1.0, 2.0 ** -7, 2.0 ** 5):
        signs = np.array([1, -1, 1])
        v = np.zeros((1, 32), np.float32)
        v[0, :3] = (signs * L * c).astype(np.float32)
        lay = oracle.Layout([3], 32)
        norms = oracle.bucket_norms(lay, v)
        assert norms[0, 0] == np.float32(s * c)
        for seed in range(20):
            codes, x, u = oracle.quantize(lay, v, norms, b, seed, 7, want_x_v=True)
            assert np.array_equal(x[0, :3], (signs * L).astype(np.float32))   # exactly on the grid
            assert np.array_equal(codes[0, :3].astype(np.int64), s + signs * L)
            assert np.all(codes[0, 3:] == s)                       # pads hold the code of 0
            q = oracle.dequantize(lay, codes[0], norms[0], b)
            assert np.array_equal(q[:3], v[0, :3].astype(np.float64))


def test_signed_zero_and_zero_norm_bucket():
    lay = oracle.Layout([64], 32)
    v = np.zeros((1, 64), np.float32)
    v[0, 1] = -0.0
    v[0, 32] = 3.0
    v[0, 33] = -4.0
    norms = oracle.bucket_norms(lay, v)
    assert norms.tolist() == [[0.0, 5.0]]
    b, s = 5, 15                            # 3/5 and 4/5 lie on levels 9 and 12
    codes = oracle.quantize(lay, v, norms, b, 11, 0)
    assert codes[0, 0] == s and codes[0, 1] == s                   # zeros of either sign: code of 0
    assert codes[0, 32] == s + 9 and codes[0, 33] == s - 12
    assert np.all(codes[0, 2:32] == s)                             # a zero-norm bucket quantizes to 0
    q = oracle.dequantize(lay, codes[0], norms[0], b)
    assert q[0] == 0 and q[1] == 0 and q[32] == 3.0 and q[33] == -4.0


def test_b1_carries_nothing():
    # b = 1: s = 0, the paper's map is undefined; reading: code 0, value 0
    lay = oracle.Layout([40], 32)
    rng = np.random.default_rng(5)
    v = rng.standard_normal((2, 64)).astype(np.float32)
    norms = oracle.bucket_norms(lay, v)
    codes = oracle.quantize(lay, v, norms, 1, 1, 1)
    assert np.all(codes == 0)
    packed = oracle.quantize_pack(lay, v, norms, 1, 1, 1)
    assert np.all(oracle.unpack_dequant_average(lay, packed, norms, 1) == 0)


def test_code_range():
    # codes live in 0 .. 2s, so they fit b bits and the all-ones pattern never occurs
    w = W.config_flat(d=4096, M=2, bucket=128, sigma=1.0)
    lay = oracle.Layout(w.segments, w.bucket)
    g = W.make_grads(w, lay.offsets, lay.D32)
    norms = oracle.bucket_norms(lay, g)
    for b in (2, 3, 8, 16):
        s = (1 << (b - 1)) - 1
        codes = oracle.quantize(lay, g, norms, b, 3, 4)
        assert codes.min() >= 0 and codes.max() <= 2 * s
        assert np.array_equal(codes > s, (g > 0) & (codes != s))   # the side of s is the sign


# --------------------------------------- brute force over all outcomes (P3 i)

@pytest.mark.parametrize("b", [2, 3, 4, 6, 9])
@pytest.mark.parametrize("d", [1, 3, 8])
def test_exact_expectation_by_enumeration(b, d):
    s = (1 << (b - 1)) - 1
    rng = np.random.default_rng(100 * b + d)
    v = np.zeros((1, 32), np.float32)
    v[0, :d] = rng.standard_normal(d).astype(np.float32) * 0.3
    lay = oracle.Layout([d], 32)
    norms = oracle.bucket_norms(lay, v)
    norm = float(norms[0, 0])
    codes, x, u = oracle.quantize(lay, v, norms, b, 42, 0, want_x_v=True)
    codes, x, u = codes[0, :d].astype(np.int64), x[0, :d].astype(np.float64), u[0, :d].astype(np.float64)
    # the oracle's position on the level grid against the definition sgn * s|g|/||g|| in fp64
    r = s * np.abs(v[0, :d].astype(np.float64)) / norm
    assert np.allclose(x, np.sign(v[0, :d]) * r, atol=4e-7 * max(1.0, s))
    sgn = np.where(x < 0, -1, 1)
    low = np.floor(np.abs(x)).astype(np.int64)                   # level l toward zero
    frac = np.abs(x) - low                                       # p_r of Eq. 6
    # the drawn code is one of the two neighbours of x, chosen by floor(x + v)
    assert np.array_equal(codes - s, np.floor(x + u).astype(np.int64))
    assert np.all(np.isin(codes - s - sgn * low, (0, 1, -1)))
    outcomes = []
    for ups in itertools.product((0, 1), repeat=d):
        ups = np.array(ups)
        p = np.prod(np.where(ups == 1, frac, 1.0 - frac))
        q = _values((s + sgn * (low + ups)).astype(np.uint32), norms[0, 0], b)
        outcomes.append((p, q))
    total = sum(p for p, _ in outcomes)
    mean = sum(p * q for p, q in outcomes)
    var = sum(p * (q - mean) ** 2 for p, q in outcomes)          # centred: no difference of large squares
    assert abs(total - 1.0) < 1e-12
    # E[Q(v)] = v up to the two fp32 roundings (each toward zero, < 1 ulp) in x = g * (s / norm)
    assert np.all(np.abs(mean - v[0, :d]) <= 2.0 ** -22 * np.abs(v[0, :d]) + 1e-30)
    # Var = (norm/s)^2 p_r (1 - p_r) per coordinate, trace <= d norm^2 / (4 s^2)
    assert np.allclose(var, (norm / s) ** 2 * frac * (1 - frac), rtol=1e-9, atol=1e-18 * (norm / s) ** 2)
    assert var.sum() <= d * norm ** 2 / (4 * s * s) * (1 + 1e-12)


# ------------------------------------------------------ Monte Carlo (P3 ii, P4)

N_WORKERS, N_STEPS = 4096, 256           # 2^20 independent draws


def _mc(v, b, seed):
    d = v.size
    lay = oracle.Layout([d], 32)
    row = np.zeros((1, 32), np.float32)
    row[0, :d] = v
    g = np.broadcast_to(row, (N_WORKERS, 32))                  # every "worker" holds the same vector
    norms = np.ascontiguousarray(np.broadcast_to(oracle.bucket_norms(lay, row), (N_WORKERS, 1)))
    s1 = np.zeros(d)
    s2 = np.zeros(d)
    for step in range(N_STEPS):
        codes = oracle.quantize(lay, g, norms, b, seed, step)
        q = _values(codes[:, :d], norms[0, 0], b)
        s1 += q.sum(0)
        s2 += (q * q).sum(0)
    n = N_WORKERS * N_STEPS
    mean = s1 / n
    return mean, s2 / n - mean * mean, float(norms[0, 0])


@pytest.mark.parametrize("b", [2, 3, 4, 8])
def test_monte_carlo_unbiased_and_variance(b):
    s = (1 << (b - 1)) - 1
    d = 16
    rng = np.random.default_rng(b)
    v = (rng.standard_normal(d) * 0.1).astype(np.float32)
    mean, var, norm = _mc(v, b, seed=2024)
    # |mean - v_j| <= 5 sigma, sigma <= (norm / 2s) / sqrt(N), N = 2^20
    tol = 5.0 * (norm / (2 * s)) / np.sqrt(N_WORKERS * N_STEPS)
    assert tol == pytest.approx(2.44e-3 * norm / s, rel=1e-2)
    assert np.all(np.abs(mean - v) <= tol)
    r = s * np.abs(v.astype(np.float64)) / norm
    f = r - np.floor(r)
    exact = (norm / s) ** 2 * (f * (1 - f)).sum()
    assert abs(var.sum() - exact) <= 0.02 * exact
    assert var.sum() <= d * norm ** 2 / (4 * s * s)            # Lemma 1


def test_variance_bound_is_attained_on_midpoints():
    # all coordinates half-way between two levels: p_r = 1/2, variance = bound
    b, s = 4, 7
    v = np.zeros(4, np.float32)
    v[:] = [3.5, 3.5, 3.5, 3.5]            # norm 7 -> r = s*3.5/7 = 3.5 exactly
    mean, var, norm = _mc(v, b, seed=7)
    assert norm == 7.0
    bound = 4 * norm ** 2 / (4 * s * s)
    assert abs(var.sum() - bound) <= 0.01 * bound
    assert np.all(np.abs(mean - v) <= 5 * (norm / (2 * s)) / 1024)


def test_average_variance_scales_as_one_over_M():
    # independent per-worker streams: Var[mean of M] = Var[single] / M
    b, s, M, steps = 4, 7, 8, 1 << 14
    rng = np.random.default_rng(3)
    d = 16
    row = np.zeros((1, 32), np.float32)
    row[0, :d] = rng.standard_normal(d) * 0.05
    lay = oracle.Layout([d], 32)
    g = np.broadcast_to(row, (M, 32))
    n1 = oracle.bucket_norms(lay, row)
    norms = np.ascontiguousarray(np.broadcast_to(n1, (M, 1)))
    s1 = np.zeros(d)
    s2 = np.zeros(d)
    for step in range(steps):
        packed = oracle.quantize_pack(lay, g, norms, b, 99, step)
        avg = oracle.unpack_dequant_average(lay, packed, norms, b)[:d].astype(np.float64)
        s1 += avg
        s2 += avg * avg
    mean = s1 / steps
    var = (s2 / steps - mean * mean).sum()
    norm = float(n1[0, 0])
    r = s * np.abs(row[0, :d].astype(np.float64)) / norm
    f = r - np.floor(r)
    single = (norm / s) ** 2 * (f * (1 - f)).sum()
    assert abs(var - single / M) <= 0.03 * single / M
    assert np.all(np.abs(mean - row[0, :d]) <= 5 * norm / (2 * s) / np.sqrt(M * steps))


# ------------------------------------------------------------ special cases (P6)

def test_b16_single_worker_is_within_one_level():
    w = W.config_flat(d=5000, M=1, bucket=512, sigma=1.0)
    lay = oracle.Layout(w.segments, w.bucket)
    g = W.make_grads(w, lay.offsets, lay.D32)
    norms = oracle.bucket_norms(lay, g)
    packed = oracle.quantize_pack(lay, g, norms, 16, 5, 0)
    out = oracle.unpack_dequant_average(lay, packed, norms, 16)
    s = 32767
    per_elem = np.repeat(norms[0], 512)[:5000] / s
    assert np.all(np.abs(out[:5000] - g[0, :5000]) <= per_elem * (1 + 1e-6))
    assert np.all(out[5000:] == 0)


def test_identical_on_level_workers_average_to_input():
    b, s = 4, 7
    row = np.zeros((1, 32), np.float32)
    row[0, :3] = [2 * 0.25, -3 * 0.25, 6 * 0.25]
    g = np.ascontiguousarray(np.broadcast_to(row, (5, 32)))
    lay = oracle.Layout([3], 32)
    norms = oracle.bucket_norms(lay, g)
    packed = oracle.quantize_pack(lay, g, norms, b, 1, 2)
    out = oracle.unpack_dequant_average(lay, packed, norms, b)
    assert np.array_equal(out, row[0])


def test_average_matches_numpy_definition():
    # (1/M) sum_m Q(g^(m)) written with numpy from the codes
    w = W.scaled_down(W.config_vgg16(M=5), 512)
    lay = oracle.Layout(w.segments, 64)
    g = W.make_grads(w, lay.offsets, lay.D32)
    norms = oracle.bucket_norms(lay, g)
    b = 6
    codes = oracle.quantize(lay, g, norms, b, 8, 3)
    packed = oracle.quantize_pack(lay, g, norms, b, 8, 3)
    for m in range(w.M):
        assert np.array_equal(oracle.unpack(packed[m], lay.D32, b), codes[m])
    out = oracle.unpack_dequant_average(lay, packed, norms, b)
    acc = np.zeros(lay.D32)
    for m in range(w.M):
        per_elem = np.zeros(lay.D32)
        for k in range(lay.nb):
            st, ln = lay.bucket_start[k], lay.bucket_len[k]
            per_elem[st: st + ln] = norms[m, k]
        s = (1 << (b - 1)) - 1
        acc += (codes[m].astype(np.float64) - s) * per_elem / s
    assert np.allclose(out, acc / w.M, rtol=1e-6, atol=1e-12)
    # the averaged quantized gradient is close to the true mean gradient:
    # per-element error below one level of the largest bucket norm
    err = np.abs(out - g.mean(0))
    assert err.max() <= norms.max() / s


# ------------------------------------------------ boundary cases of Eq. 6

def test_rounding_boundaries():
    # With s = 1 and a norm of exactly 1 the position on the grid is the input itself,
    # and the drawn v of every element is known.  The level goes up (away from zero)
    # exactly when p_r + v >= 1 for positive inputs and v < p_r for negative ones.
    lay = oracle.Layout([32], 32)
    one = np.ones((1, 1), np.float32)
    zeros = np.zeros((1, 32), np.float32)
    _, _, v = oracle.quantize(lay, zeros, one, 2, 77, 5, want_x_v=True)
    v = v[0]
    assert np.all((v > 0) & (v < 1))
    s = 1
    cases = [
        (np.float32(1.0) - v, s + 1),                              # p_r + v = 1: up
        (np.nextafter(np.float32(1.0) - v, np.float32(0)), s),     # just below: stays
        (-v, s),                                                   # v = p_r: stays at 0
        (np.nextafter(-v, np.float32(-1)), s - 1),                 # v < p_r: goes to -1
        (zeros[0], s), (np.full(32, 1.0, np.float32), s + 1), (np.full(32, -1.0, np.float32), s - 1),
    ]
    for g, want in cases:
        g = np.ascontiguousarray(g.astype(np.float32).reshape(1, 32))
        codes, x, v2 = oracle.quantize(lay, g, one, 2, 77, 5, want_x_v=True)
        assert np.array_equal(x, g) and np.array_equal(v2[0], v)
        assert np.all(codes[0] == want)


def test_position_is_rounded_toward_zero_and_never_leaves_the_grid():
    # x = RZ(g * RZ(s / norm)): never beyond the exact s*g/norm, hence |x| <= s whenever
    # |g| <= norm, with no clamp; a bucket of one element is the extreme case |g| = norm
    rng = np.random.default_rng(11)
    for b in (3, 4, 7, 16):
        s = (1 << (b - 1)) - 1
        w = W.config_flat(d=2048, M=2, bucket=64, sigma=1.0, seed=b)
        lay = oracle.Layout(w.segments, w.bucket)
        g = W.make_grads(w, lay.offsets, lay.D32)
        norms = oracle.bucket_norms(lay, g)
        codes, x, _ = oracle.quantize(lay, g, norms, b, 3, 1, want_x_v=True)
        exact = s * g.astype(np.float64) / np.repeat(norms.astype(np.float64), 64, axis=1)
        assert np.all(np.abs(x) <= np.abs(exact)) and np.all(np.sign(x) * np.sign(exact) >= 0)
        assert np.all(np.abs(x - exact) <= 2.0 ** -22 * np.abs(exact))          # two roundings, each < 1 ulp
        assert np.mean(np.abs(x) < np.abs(exact)) > 0.5                          # and it really is toward zero
        assert codes.max() <= 2 * s
        a = rng.uniform(0.5, 2.0, 2000).astype(np.float32)
        lay1 = oracle.Layout([1], 32)
        for val in a[:64]:
            for sign in (1.0, -1.0):
                g1 = np.zeros((1, 32), np.float32)
                g1[0, 0] = sign * val
                n1 = oracle.bucket_norms(lay1, g1)
                assert n1[0, 0] == val
                codes1, x1, _ = oracle.quantize(lay1, g1, n1, b, 5, 0, want_x_v=True)
                assert abs(x1[0, 0]) <= s and abs(x1[0, 0]) >= s * (1 - 2.0 ** -22)
                assert 0 <= codes1[0, 0] <= 2 * s
