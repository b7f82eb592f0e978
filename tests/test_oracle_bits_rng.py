"""Pins for the oracle's bit rule (Eq. 17) and its Philox generator (CPU only)."""
import math

import numpy as np
import pytest

import oracle
from conftest import read_golden


def _norms_with_gbar(gbar, M=3, nb=5):
    """Bucket norms whose G-bar (root mean over workers of squared vector norms) is gbar."""
    n = np.zeros((M, nb), np.float32)
    n[:, 0] = gbar              # each worker's vector norm is gbar -> mean square gbar^2
    return n


# --------------------------------------------------------- hand-worked cases (P5)

@pytest.mark.parametrize("gbar,b_want", [
    (1.0, 2),        # x = 1 -> s >= 1 -> b = 2
    (3.0, 3),        # x = 3 -> s = 3
    (3.0001, 4),     # just above a threshold -> next b
    (7.0, 4),
    (127.0, 8),
    (0.0, 2),        # clamped to b_min
    (1e9, 16),       # clamped to b_max
])
def test_bit_rule_hand_cases(gbar, b_want):
    # T = eps_hat makes sqrt(T/eps_hat) = 1 and t = T-1 makes the alpha factor 1: x = G-bar
    b, s, x = oracle.choose_bits(_norms_with_gbar(gbar), T=50, t=49, eps_hat=50.0, alpha=0.9)
    assert x == pytest.approx(gbar, rel=1e-6)
    assert b == b_want and s == (1 << (b - 1)) - 1


def test_gbar_is_mean_over_workers_of_squared_norms():
    # workers with vector norms 3 and 4 (spread over several buckets): G-bar^2 = (9 + 16)/2
    n = np.zeros((2, 4), np.float32)
    n[0, :] = [1, 2, 2, 0]            # 1+4+4 = 9
    n[1, :] = [0, 0, 4, 0]
    b, s, x = oracle.choose_bits(n, T=10, t=9, eps_hat=10.0, alpha=0.5)
    assert x == pytest.approx(math.sqrt(12.5), rel=1e-12)


def test_fixed_b_bypasses_rule():
    for fb in (1, 2, 9, 16):
        b, s, _ = oracle.choose_bits(_norms_with_gbar(100.0), 10, 0, 1.0, 0.9, fixed_b=fb)
        assert b == fb and s == (1 << (fb - 1)) - 1


def test_closed_form_and_budget():
    # Eq. 17 solves the constraint of Eq. 16 with equal spending per step:
    # alpha^(T-1-t) G_t^2 / (2^(b*-1) - 1)^2 = eps_hat / T for the real-valued b*.
    T, alpha, eps_hat = 40, 0.93, 0.37
    rng = np.random.default_rng(0)
    spent = 0.0
    for t in range(T):
        gbar = float(rng.uniform(0.5, 20.0))
        b, s, x = oracle.choose_bits(_norms_with_gbar(gbar), T, t, eps_hat, alpha, b_min=2, b_max=24)
        gb = float(np.float32(gbar))
        b_star = math.log2(math.sqrt(T / eps_hat) * alpha ** ((T - 1 - t) / 2) * gb + 1) + 1
        assert math.log2(x + 1) + 1 == pytest.approx(b_star, rel=1e-12)
        assert alpha ** (T - 1 - t) * gb ** 2 / (2 ** (b_star - 1) - 1) ** 2 == pytest.approx(eps_hat / T, rel=1e-9)
        # integer b = ceiling of b* (smallest b whose s >= x)
        assert b == max(2, math.ceil(b_star - 1e-12))
        spent += alpha ** (T - 1 - t) * gb ** 2 / s ** 2
    assert spent <= eps_hat * (1 + 1e-12)       # ceiling keeps the quantization-error budget


def test_monotone_in_gbar_t_and_budget():
    T, alpha = 30, 0.9
    prev = 0
    for gbar in np.geomspace(0.01, 1e4, 60):
        b, _, _ = oracle.choose_bits(_norms_with_gbar(float(gbar)), T, 10, 1.0, alpha)
        assert b >= prev
        prev = b
    prev = 0
    for t in range(T):
        b, _, _ = oracle.choose_bits(_norms_with_gbar(5.0), T, t, 1.0, alpha)
        assert b >= prev
        prev = b
    prev = 0
    for eps in np.geomspace(100.0, 1e-4, 40):
        b, _, _ = oracle.choose_bits(_norms_with_gbar(5.0), T, 10, float(eps), alpha)
        assert b >= prev
        prev = b


@pytest.mark.parametrize("rho,direction", [(0.80, -1), (0.99, +1)])
def test_trend_criterion(rho, direction):
    # Sec. V-C: with G_{t+1}/G_t = rho, x_t moves by rho/sqrt(alpha) per step:
    # bits fall when rho < sqrt(alpha) and rise when rho > sqrt(alpha)
    T, alpha = 60, 0.9 ** 2            # sqrt(alpha) = 0.9
    xs, bs = [], []
    for t in range(T):
        b, _, x = oracle.choose_bits(_norms_with_gbar(50.0 * rho ** t), T, t, 1e-3, alpha, b_max=16)
        xs.append(x)
        bs.append(b)
    ratios = np.array(xs[1:]) / np.array(xs[:-1])
    assert np.allclose(ratios, rho / 0.9, rtol=1e-5)
    steps = np.diff(bs)
    assert np.all(steps * direction >= 0) and bs[-1] * direction > bs[0] * direction


# ---------------------------------------------------------------- Philox (P7)

def test_philox_known_answers():
    for row in read_golden("philox4x32_10_kat.txt"):
        v = [int(x, 16) for x in row]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [hex(x) for x in out] == [hex(x) for x in v[6:10]]


def test_philox_counter_and_key_separation():
    base = oracle.philox4x32_10([5, 0, 2, 3], [7, 9])
    for i in range(4):
        c = [5, 0, 2, 3]
        c[i] += 1
        assert not np.array_equal(oracle.philox4x32_10(c, [7, 9]), base)
    assert not np.array_equal(oracle.philox4x32_10([5, 0, 2, 3], [8, 9]), base)
    assert not np.array_equal(oracle.philox4x32_10([5, 0, 2, 3], [7, 10]), base)


def test_uniform_is_philox_half_word_of_the_element():
    # element j of worker m at a step draws from the block with counter (j >> 3, 0, m, step)
    # and key (seed lo, seed hi): half (j & 1) of word ((j >> 1) & 3), low half first;
    # with k that 16-bit value, v = (2k + 1) / 2^17
    lay = oracle.Layout([64], 32)
    g = np.ones((3, 64), np.float32)
    norms = oracle.bucket_norms(lay, g)
    seed, step = (0xDEADBEEF << 32) | 0x12345678, 77
    _, _, v = oracle.quantize(lay, g, norms, 4, seed, step, want_x_v=True)
    for m in range(3):
        for j in (0, 1, 2, 5, 7, 8, 31, 32, 63):
            blk = oracle.philox4x32_10([j >> 3, 0, m, step], [0x12345678, 0xDEADBEEF])
            word = int(blk[(j >> 1) & 3])
            k = (word >> 16) if (j & 1) else (word & 0xFFFF)
            assert float(v[m, j]) == (2 * k + 1) / 2.0 ** 17


def test_uniform_statistics():
    # 2^22 draws: mean 1/2 within 5 sigma, chi-square over 256 cells, in (0,1)
    lay = oracle.Layout([1 << 20], 4096)
    g = np.ones((4, 1 << 20), np.float32)
    norms = oracle.bucket_norms(lay, g)
    _, _, u = oracle.quantize(lay, g, norms, 4, 123, 0, want_x_v=True)
    u = u.ravel().astype(np.float64)
    n = u.size
    assert u.min() > 0.0 and u.max() < 1.0
    assert np.all((u * 2 ** 17) % 2 == 1)                   # odd multiples of 2^-17: the midpoint grid
    assert abs(u.mean() - 0.5) < 5 * math.sqrt(1 / 12 / n)
    counts = np.bincount((u * 256).astype(np.int64), minlength=256)
    chi2 = ((counts - n / 256) ** 2 / (n / 256)).sum()
    assert chi2 < 255 + 5 * math.sqrt(2 * 255)
    # rows (workers) are different streams
    assert not np.array_equal(u[: 1 << 20], u[1 << 20: 2 << 20])
    assert abs(np.corrcoef(u[: 1 << 20], u[1 << 20: 2 << 20])[0, 1]) < 5 / math.sqrt(1 << 20)
