"""Host side of Algorithm 1's bit-width updates.

The kernels take a ``dq.Rule`` per call; this module decides which rule a training loop
passes at iteration t: Eq. 17 with the contraction rate alpha either given or estimated
from the losses as Sec. V-C proposes, refreshed every ``tau`` iterations (Algorithm 1
recomputes b "every tau iterations").  Nothing here touches the device.
"""
from __future__ import annotations

from typing import Optional

from . import dq


def alpha_est(F_t: float, F_0: float, t: int) -> float:
    """Sec. V-C: alpha_est = (F(x_t) / F(x_0))^(1/t), with F(x*) taken as 0."""
    if t < 1:
        raise ValueError("the estimate needs at least one iteration")
    if not (F_0 > 0.0 and F_t > 0.0):
        raise ValueError("losses must be positive")
    return (F_t / F_0) ** (1.0 / t)


class BitSchedule:
    """Which bit rule applies at iteration t.

    ``T``, ``eps_hat``: horizon and error budget of Eq. 16/17.  ``alpha``: the contraction
    rate if known; otherwise ``observe`` feeds losses and the estimate of Sec. V-C is used
    (until the first observation the schedule holds ``b0``).  ``tau``: the bit width is
    re-derived at iterations 0, tau, 2 tau, ...; in between the last b is kept.
    """

    def __init__(self, T: int, eps_hat: float, tau: int = 1, alpha: Optional[float] = None, b0: int = 4,
                 b_min: int = 2, b_max: int = 16):
        if T < 1 or tau < 1 or not eps_hat > 0.0:
            raise ValueError("T >= 1, tau >= 1 and eps_hat > 0 are required")
        self.T, self.eps_hat, self.tau, self.alpha = int(T), float(eps_hat), int(tau), alpha
        self.b0, self.b_min, self.b_max = int(b0), int(b_min), int(b_max)
        self._F0 = None
        self._alpha_est = None

    def observe(self, t: int, loss: float) -> None:
        """Loss F(x_t) as the training loop sees it; t = 0 sets the reference F(x_0)."""
        if t == 0:
            self._F0 = float(loss)
        elif self._F0 is not None:
            # the estimate can exceed 1 while the loss still rises; Eq. 17 needs alpha in (0, 1]
            self._alpha_est = min(1.0, alpha_est(float(loss), self._F0, t))

    def due(self, t: int) -> bool:
        """True at the iterations where b is re-derived from the norms."""
        return t % self.tau == 0

    def current_alpha(self) -> Optional[float]:
        return self.alpha if self.alpha is not None else self._alpha_est

    def rule(self, t: int) -> Optional[dq.Rule]:
        """Rule for iteration t (0 <= t < T), or None where the previous b stays in force."""
        if not 0 <= t < self.T:
            raise ValueError("t outside the horizon")
        if not self.due(t):
            return None
        a = self.current_alpha()
        if a is None:
            return dq.Rule.fixed(self.b0)
        return dq.Rule.dynamic(self.T, t, self.eps_hat, a, self.b_min, self.b_max)
