"""Oracle of the spatial controller (TEST INFRASTRUCTURE ONLY; nothing on the product path imports this).

Plain Python restatement of the paper's bandwidth-guided SM throttling (Sec. 4.3, Eq. 1; Algorithm 1
step 3) and of the offline choice of the co-running cap from a fixed-SM sweep (Sec. 4.1).  It shares no
code with the library's controller; the tests compare the two decision by decision.

Readings where the paper is silent (the same ones the C header states): the moving average is
Bhat <- gamma * B + (1 - gamma) * Bhat with Bhat = B on the first sample and is updated on every step;
snap takes the nearest ladder value, the lower one on a tie; delta_step counts SMs.

Parity status: the paper prints no worked example of the controller (its Fig. 10 is a plot), so paper-level
parity is unpinned; the definition is pinned by closed forms and invariants in tests/test_control.py.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple


class SpatialOracle:
    def __init__(self, s_total: int, s_aggr: int, ladder: Sequence[int], b_sat: float, gamma: float,
                 delta_step: int):
        self.s_total, self.s_aggr = s_total, s_aggr
        self.ladder: List[int] = list(ladder)
        self.b_sat, self.gamma, self.delta_step = b_sat, gamma, delta_step
        self.bhat: Optional[float] = None
        self.s_shared = s_aggr

    def snap(self, target: float) -> int:
        """Nearest ladder value; on a tie the lower one."""
        best = self.ladder[0]
        for level in self.ladder[1:]:
            if abs(level - target) < abs(best - target):
                best = level
        return best

    def update(self, downstream_active: bool, pressure: float) -> Tuple[int, int]:
        # Sec. 4.3, "Bandwidth-pressure signal": smoothed with an EWMA of weight gamma
        self.bhat = pressure if self.bhat is None else self.gamma * pressure + (1.0 - self.gamma) * self.bhat
        if not downstream_active:
            # Eq. 1, first case; Algorithm 1 step 3: applied whenever the downstream stages are inactive
            self.s_shared = self.s_aggr
        else:
            # Eq. 1, second case: rho = clamp(Bhat / B_sat, 0, 1), position inside [S_min, S_cap], snapped
            rho = min(max(self.bhat / self.b_sat, 0.0), 1.0)
            s_min, s_cap = self.ladder[0], self.ladder[-1]
            s_star = self.snap(s_min + rho * (s_cap - s_min))
            # Sec. 4.3: during co-running the cap stays within the ladder, "never back to full allocation"
            # (S_cap < S_aggr), so a cap above S_cap left by the inactive case is replaced at once; the
            # hysteresis (keep the previous cap unless the level moves by at least delta_step) acts only
            # between ladder levels
            if self.s_shared > s_cap or abs(s_star - self.s_shared) >= self.delta_step:
                self.s_shared = s_star
        # "Complementary downstream headroom"
        return self.s_shared, max(0, self.s_total - self.s_shared)


def derive_cap(budgets: Sequence[int], latency: Sequence[float], s_total: int, tolerance: float) -> int:
    """Sec. 4.1: the smallest SM count that reaches near-best latency.  Full allocation is not a candidate
    (co-running must leave headroom, Sec. 3.2), so "best" is the best among the budgets below s_total."""
    below = [(b, t) for b, t in zip(budgets, latency) if b < s_total]
    best = min(t for _, t in below)
    return min(b for b, t in below if t <= best * (1.0 + tolerance))
