"""Host logic of the bit-width schedule (Algorithm 1's tau-periodic refresh, alpha_est of Sec. V-C)."""
import pytest

from paper_2107_14575_b200 import schedule


def test_alpha_est_recovers_a_geometric_rate():
    for alpha in (0.5, 0.9, 0.999):
        for t in (1, 7, 100):
            assert schedule.alpha_est(3.0 * alpha ** t, 3.0, t) == pytest.approx(alpha, rel=1e-12)
    with pytest.raises(ValueError):
        schedule.alpha_est(1.0, 1.0, 0)
    with pytest.raises(ValueError):
        schedule.alpha_est(-1.0, 1.0, 3)


def test_refresh_every_tau_and_fixed_start():
    s = schedule.BitSchedule(T=20, eps_hat=2.0, tau=5, b0=6)
    assert [t for t in range(20) if s.due(t)] == [0, 5, 10, 15]
    assert s.rule(3) is None
    r0 = s.rule(0)
    assert r0.fixed_b == 6                      # no alpha known yet: the initial b
    s.observe(0, 8.0)
    s.observe(5, 8.0 * 0.9 ** 5)
    r5 = s.rule(5)
    assert r5.fixed_b == 0 and r5.T == 20 and r5.t == 5 and r5.eps_hat == 2.0
    assert r5.alpha == pytest.approx(0.9)
    s.observe(10, 100.0)                        # a loss above F(x_0): the estimate is capped at 1
    assert s.rule(10).alpha == 1.0
    with pytest.raises(ValueError):
        s.rule(20)


def test_given_alpha_wins_over_the_estimate():
    s = schedule.BitSchedule(T=10, eps_hat=1.0, alpha=0.8)
    s.observe(0, 1.0)
    s.observe(3, 0.1)
    r = s.rule(3)
    assert r.alpha == 0.8 and (r.b_min, r.b_max) == (2, 16)
    with pytest.raises(ValueError):
        schedule.BitSchedule(T=0, eps_hat=1.0)
