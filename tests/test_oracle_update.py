"""Pins of the oracle's parameter update (Eq. 2; Algorithm 1, "Update the global parameters").

What fixes it independently of its own code:
  * exact arithmetic: identical workers whose entries sit on levels average to the entries
    themselves, so x - eta * v must come out exactly (catches a wrong sign, a dropped 1/M, eta
    applied twice);
  * gradient descent on the isotropic quadratic of Sec. V-B: with exact gradients lambda (x - x*)
    quantized at 16 bits the iterates contract as (1 - eta lambda)^t up to the quantizer's level
    spacing -- with "+ eta" (as one sentence of the paper prints it) they would grow instead;
  * padding and the degenerate cases (eta = 0, b = 1) leave x as it is.
"""
import numpy as np

import oracle


def _round(lay, g, b, seed, step):
    norms = oracle.bucket_norms(lay, g)
    return norms, oracle.quantize_pack(lay, g, norms, b, seed, step)


def test_on_level_identical_workers_update_exactly():
    lay = oracle.Layout([64], 32)
    b = 4                                   # s = 7; (2, 3, 6) has norm 7
    row = np.zeros(64, np.float32)
    row[:3] = [2 * 0.25, -3 * 0.25, 6 * 0.25]
    row[32:35] = [-6.0, 2.0, 3.0]
    g = np.ascontiguousarray(np.broadcast_to(row, (4, 64)))
    norms, packed = _round(lay, g, b, 1, 2)
    x = np.arange(64, dtype=np.float32) * 0.125 - 3.0
    for eta in (0.5, 0.25, 2.0):
        got = oracle.unpack_average_update(lay, packed, norms, b, eta, x)
        assert np.array_equal(got, (x - np.float32(eta) * row).astype(np.float32))
    # eta = 0 and a negative eta (ascent) behave as the formula says
    assert np.array_equal(oracle.unpack_average_update(lay, packed, norms, b, 0.0, x), x)
    assert np.array_equal(oracle.unpack_average_update(lay, packed, norms, b, -0.5, x), x + np.float32(0.5) * row)


def test_padding_and_one_bit_leave_x_alone():
    lay = oracle.Layout([5, 40, 0, 33], 32)
    rng = np.random.default_rng(3)
    g = np.zeros((3, lay.D32), np.float32)
    for i, n in enumerate([5, 40, 0, 33]):
        g[:, lay.offsets[i]: lay.offsets[i] + n] = rng.normal(size=(3, n)).astype(np.float32)
    x = rng.normal(size=lay.D32).astype(np.float32)
    norms, packed = _round(lay, g, 6, 9, 0)
    got = oracle.unpack_average_update(lay, packed, norms, 6, 0.1, x)
    valid = np.zeros(lay.D32, bool)
    for i, n in enumerate([5, 40, 0, 33]):
        valid[lay.offsets[i]: lay.offsets[i] + n] = True
    assert np.array_equal(got[~valid], x[~valid])
    assert np.all(got[valid] != x[valid])
    # the update is the average scaled by -eta (fp64 evaluation of both sides)
    avg = oracle.unpack_dequant_average(lay, packed, norms, 6).astype(np.float64)
    np.testing.assert_allclose(got[valid], x[valid] - 0.1 * avg[valid], rtol=0, atol=2e-7)
    # b = 1: s = 0, every value 0
    norms1, packed1 = _round(lay, g, 1, 9, 0)
    assert np.array_equal(oracle.unpack_average_update(lay, packed1, norms1, 1, 0.1, x), x)


def test_quadratic_contracts_at_the_rate_of_gradient_descent():
    d, M, b, lam, eta, T = 2048, 4, 16, 2.0, 0.15, 30
    s = (1 << (b - 1)) - 1
    lay = oracle.Layout([d], 512)
    rng = np.random.default_rng(11)
    x_star = rng.normal(size=d)
    x0 = x_star + rng.normal(size=d) * 3.0
    x = x0.astype(np.float32)
    rho = 1.0 - eta * lam
    slack = 0.0
    for t in range(T):
        grad = (lam * (x.astype(np.float64) - x_star)).astype(np.float32)
        g = np.ascontiguousarray(np.broadcast_to(grad, (M, d)))
        norms, packed = _round(lay, g, b, 5, t)
        x = oracle.unpack_average_update(lay, packed, norms, b, eta, x)
        # each step may be off by eta times one level of the bucket, plus fp32 rounding of x and of the gradient
        slack = abs(rho) * slack + eta * float(norms.max()) / s + 4e-7 * (1 + eta * lam) * float(np.abs(x).max() + np.abs(x_star).max())
        want = x_star + rho ** (t + 1) * (x0 - x_star)
        assert np.max(np.abs(x - want)) <= slack + 1e-6, (t, np.max(np.abs(x - want)), slack)
    assert np.linalg.norm(x - x_star) < 1e-3 * np.linalg.norm(x0 - x_star)
