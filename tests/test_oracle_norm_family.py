"""Pins for the other members of the quantizer family of Eq. 5 (CPU only): the
l_infinity norm, and one norm per tensor (the paper's own normalisation, a bucket
as large as the vector).

What fixes the expected values: numpy's max and norm; the fact that the entry of
largest magnitude sits exactly on the outermost level s and is therefore
reproduced for every draw; Lemma 1 (unbiasedness and the trace bound
d * ||g||_p^2 / (4 s^2), whose proof uses only |g_j| <= ||g||_p) checked by
brute force over every rounding outcome.
"""
import itertools

import numpy as np
import pytest

import oracle
from paper_2107_14575_b200 import workloads as W


def test_linf_norms_are_numpy_max_abs():
    w = W.scaled_down(W.config_resnet18(M=3), 64)
    lay = oracle.Layout(w.segments, 96)                          # ragged buckets, several tensors
    g = W.make_grads(w, lay.offsets, lay.D32, pad_value=1e30)    # pads must be ignored
    norms = oracle.bucket_norms(lay, g, oracle.NORM_LINF)
    for m in range(w.M):
        for k in range(lay.nb):
            st, ln = lay.bucket_start[k], lay.bucket_len[k]
            assert norms[m, k] == np.max(np.abs(g[m, st: st + ln]))       # exact: no arithmetic
    # l_inf <= l_2 <= sqrt(n) * l_inf for every bucket
    n2 = oracle.bucket_norms(lay, g).astype(np.float64)
    ni = norms.astype(np.float64)
    assert np.all(ni <= n2 * (1 + 1e-6))
    assert np.all(n2 <= np.sqrt(lay.bucket_len)[None, :] * ni * (1 + 1e-6))


def test_linf_special_values():
    lay = oracle.Layout([64, 5], 32)
    g = np.zeros((1, lay.D32), np.float32)
    g[0, 3] = -7.5
    g[0, 40] = np.nan
    g[0, 41] = 100.0
    g[0, 64] = -0.0
    n = oracle.bucket_norms(lay, g, oracle.NORM_LINF)[0]
    assert n[0] == 7.5                      # sign is dropped
    assert np.isnan(n[1])                   # a NaN entry is not skipped by the max
    assert n[2] == 0.0 and not np.signbit(n[2])
    g[0, 41] = np.inf
    g[0, 40] = 1.0
    assert np.isinf(oracle.bucket_norms(lay, g, oracle.NORM_LINF)[0, 1])


def test_whole_tensor_bucket_is_one_norm_per_tensor():
    segs = [1000, 33, 0, 5000, 1]
    bucket = oracle.whole_tensor_bucket(segs)
    assert bucket % 32 == 0 and bucket >= max(segs)
    lay = oracle.Layout(segs, bucket)
    assert lay.nb == 4                                           # the empty tensor has no bucket
    rng = np.random.default_rng(7)
    g = rng.standard_normal((2, lay.D32)).astype(np.float32)
    n2 = oracle.bucket_norms(lay, g)
    ni = oracle.bucket_norms(lay, g, oracle.NORM_LINF)
    k = 0
    for o, n in zip(lay.offsets, segs):
        if n == 0:
            continue
        for m in range(2):
            t = g[m, o: o + n].astype(np.float64)
            assert abs(n2[m, k] - np.linalg.norm(t)) <= 1e-7 * np.linalg.norm(t)
            assert ni[m, k] == np.max(np.abs(g[m, o: o + n]))
        k += 1


@pytest.mark.parametrize("b", [2, 3, 5, 8, 16])
def test_linf_largest_entry_is_reproduced_for_every_draw(b):
    """With the l_inf norm the largest entry has |g| / norm = 1: it lies on level s,
    p_r = 0, and Eq. 6 must return it whatever the uniform is.  Codes stay in 0..2s."""
    s = (1 << (b - 1)) - 1
    rng = np.random.default_rng(b)
    lay = oracle.Layout([200], 64)
    g = np.zeros((1, lay.D32), np.float32)
    g[0, :200] = rng.standard_normal(200).astype(np.float32) * 3e-3
    norms = oracle.bucket_norms(lay, g, oracle.NORM_LINF)
    for step in range(20):
        codes = oracle.quantize(lay, g, norms, b, 99, step)[0]
        assert codes.max() <= 2 * s
        for k in range(lay.nb):
            st, ln = lay.bucket_start[k], lay.bucket_len[k]
            j = st + int(np.argmax(np.abs(g[0, st: st + ln])))
            assert codes[j] == (2 * s if g[0, j] > 0 else 0)
            val = (float(codes[j]) - s) * float(norms[0, k]) / s
            assert val == float(g[0, j])


@pytest.mark.parametrize("p", [oracle.NORM_L2, oracle.NORM_LINF])
@pytest.mark.parametrize("b", [2, 4, 7])
def test_lemma1_by_enumeration_for_both_norms(p, b):
    """E[Q(g)] = g and Tr Var <= d ||g||_p^2 / (4 s^2) over all 2^d outcomes, d = 6."""
    d = 6
    s = (1 << (b - 1)) - 1
    rng = np.random.default_rng(10 * b + p)
    v = np.zeros((1, 32), np.float32)
    v[0, :d] = rng.standard_normal(d).astype(np.float32)
    lay = oracle.Layout([d], 32)
    norms = oracle.bucket_norms(lay, v, p)
    norm = float(norms[0, 0])
    _, x, _ = oracle.quantize(lay, v, norms, b, 5, 0, want_x_v=True)
    x = x[0, :d].astype(np.float64)
    assert np.all(np.abs(x) <= s)                                # never leaves the grid
    assert np.allclose(x, s * v[0, :d].astype(np.float64) / norm, atol=4e-7 * s)
    sgn = np.where(x < 0, -1.0, 1.0)
    low = np.floor(np.abs(x))
    frac = np.abs(x) - low
    mean = np.zeros(d)
    second = np.zeros(d)
    for ups in itertools.product((0, 1), repeat=d):
        ups = np.array(ups)
        prob = np.prod(np.where(ups == 1, frac, 1.0 - frac))
        q = sgn * (low + ups) * norm / s
        mean += prob * q
        second += prob * q * q
    var = second - mean * mean
    assert np.all(np.abs(mean - v[0, :d]) <= 2.0 ** -22 * np.abs(v[0, :d]) + 1e-30)
    assert var.sum() <= d * norm ** 2 / (4 * s * s) * (1 + 1e-12)
    if p == oracle.NORM_LINF:
        # the l_inf grid is finer than the l_2 grid of the same vector: smaller variance bound
        n2 = float(oracle.bucket_norms(lay, v)[0, 0])
        assert norm <= n2


def test_whole_tensor_quantizer_matches_the_definition():
    """One norm per tensor, tensors longer than any bucketed layout allows: the value of
    every element is within one level step of the input and the mean error is small."""
    segs = [9000, 70]
    lay = oracle.Layout(segs, oracle.whole_tensor_bucket(segs))
    rng = np.random.default_rng(3)
    g = np.zeros((1, lay.D32), np.float32)
    for o, n in zip(lay.offsets, segs):
        g[0, o: o + n] = rng.standard_normal(n).astype(np.float32)
    b = 9
    s = (1 << (b - 1)) - 1
    for p in (oracle.NORM_L2, oracle.NORM_LINF):
        norms = oracle.bucket_norms(lay, g, p)
        codes = oracle.quantize(lay, g, norms, b, 1, 2)
        packed = oracle.pack(codes[0], b)[None, :]
        out = oracle.unpack_dequant_average(lay, packed, norms, b)
        for k, (o, n) in enumerate(zip(lay.offsets, segs)):
            step = float(norms[0, k]) / s
            err = out[o: o + n].astype(np.float64) - g[0, o: o + n]
            assert np.max(np.abs(err)) <= step * (1 + 1e-6)
            assert abs(err.mean()) <= 5 * step / 2 / np.sqrt(n)
