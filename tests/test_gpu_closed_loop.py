"""Closed loop on the GPU: Algorithm 1 on the isotropic quadratic of Sec. V-B.

F(x) = lambda/2 |x - x*|^2, every worker holds the exact gradient lambda (x - x*), so the only
noise is the quantizer's.  The whole chain runs through the library (norms, Eq. 5/6, packing,
average, the update of Eq. 2, the bit rule of Eq. 17 on the device); the test then checks the
trajectory against what the paper derives:
  * Theorem 3 in its isotropic form: F(x_T) - F* = beta^T (F(x_0) - F*) + lambda eta^2 / 2 *
    sum_t beta^(T-1-t) Tr Sigma_t, with Tr Sigma_t the exact variance of Lemma 1's proof,
    (1/M) sum_k (norm_k / s)^2 sum_j p_j (1 - p_j), evaluated on the trajectory itself; what
    is left is a martingale term whose standard deviation the test computes;
  * the constraint of Eq. 16 that Eq. 17 is built to meet: sum_t alpha^(T-1-t) G_t^2 / s_t^2 <= eps_hat;
  * Sec. V-D: when the gradient norm shrinks exactly as sqrt(alpha) per step, b stays constant.
"""
import numpy as np
import pytest
import torch

from paper_2107_14575_b200 import dq, schedule
from paper_2107_14575_b200.pipeline import Round

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib(dqlib):
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")


@pytest.mark.parametrize("p,b0,x_first", [("l2", 5, 9.0), ("linf", 3, 2.0)])
def test_quadratic_follows_theorem_3_and_the_error_budget(p, b0, x_first):
    """l2: per-bucket l_2 norms, b = 5.  linf: the l_inf member of the family at b = 3 (its level
    grid is ~sqrt(bucket) / 3.5 times finer, so a coarser b keeps the quantizer's share of F_T well
    above the test's resolution); Lemma 1's variance formula is the same for both."""
    d, bucket, M, lam, eta, T = 1 << 16, 512, 4, 1.0, 0.2, 30
    rho = 1.0 - eta * lam
    beta = rho * rho                                   # contraction of F per step: the alpha of Eq. 17
    rng = np.random.default_rng(2107)
    x_star = rng.normal(size=d)
    x0 = x_star + rng.normal(size=d)
    xs = torch.from_numpy(x_star.astype(np.float32)).cuda()
    x = torch.from_numpy(x0.astype(np.float32)).cuda()

    rnd = Round([d], bucket, M, norm=dq.NORM_L2 if p == "l2" else dq.NORM_LINF)
    g0 = lam * (x0 - x_star)
    if p == "l2":
        G0sq = float((g0 ** 2).sum())                  # (1/M) sum_m sum_k norm^2 with M identical workers
    else:
        G0sq = float((np.abs(g0).reshape(-1, bucket).max(axis=1) ** 2).sum())
    # Eq. 17: x = x_first at t = 0 and x_first / sqrt(alpha) when step t + 1 is sized from step t's norms
    # (9 -> 11.25: b = 5, s = 15; 2 -> 2.5: b = 3, s = 3)
    eps_hat = T * beta ** (T - 1) * G0sq / x_first ** 2
    sched = schedule.BitSchedule(T, eps_hat, tau=1, alpha=beta, b0=b0)
    rnd.bits_(dq.Rule.fixed(b0))

    def F(xt):
        return 0.5 * lam * float(((xt.double() - xs.double()) ** 2).sum())

    F0 = F(x)
    bits, budget, noise_term, var_FT = [], 0.0, 0.0, 0.0
    for t in range(T):
        b = rnd.bits()
        s = (1 << (b - 1)) - 1
        bits.append(b)
        grad = lam * (x - xs)
        grads = grad.unsqueeze(0).expand(M, d).contiguous()
        nxt = sched.rule(t + 1) if t + 1 < T else dq.Rule.fixed(b)
        err_before = (x.double() - xs.double()).cpu().numpy()
        rnd.step_fused(grads, nxt, 99, t, params=x, lr=eta)
        torch.cuda.synchronize()
        assert rnd.read_status() == 0
        # exact variance of the averaged quantized gradient (Lemma 1's proof, per element), from this step's data
        norms = rnd.norms[0].double().cpu().numpy()                 # identical for all workers
        gh = grad.double().cpu().numpy().reshape(-1, bucket)
        pos = s * np.abs(gh) / norms[:, None]
        p = pos - np.floor(pos)
        var_j = (norms[:, None] / s) ** 2 * p * (1.0 - p) / M       # variance of each averaged entry
        tr_sigma = float(var_j.sum())
        w = beta ** (T - 1 - t)
        noise_term += 0.5 * lam * eta * eta * w * tr_sigma
        # martingale part of F_T: the cross term lambda rho eta (x_t - x*) . eps_t and the centred square
        var_FT += w * w * ((lam * rho * eta) ** 2 * float((err_before.reshape(-1, bucket) ** 2 * var_j).sum())
                           + (0.5 * lam * eta * eta) ** 2 * 2.0 * float((var_j ** 2).sum()))
        budget += w * float((norms ** 2).sum()) / s ** 2
    FT = F(x)

    pred = beta ** T * F0 + noise_term
    sigma = np.sqrt(var_FT)
    assert noise_term > 10.0 * sigma                   # the quantizer's share is far above the test's resolution
    assert abs(FT - pred) <= 6.0 * sigma + 1e-5 * pred, (FT, pred, sigma)
    assert budget <= eps_hat * (1.0 + 1e-9)
    assert bits == [b0] * T                            # the norm falls as sqrt(alpha): constant b
