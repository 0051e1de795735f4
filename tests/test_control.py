"""The spatial controller (Sec. 4.3, Eq. 1; Algorithm 1 step 3) and the cap derivation (Sec. 4.1).

First the oracle is pinned against what the paper and the arithmetic fix (closed forms, invariants); then the
library's controller is compared with the oracle decision by decision on seeded random streams."""
import math

import numpy as np
import pytest

from oracle.control import SpatialOracle, derive_cap

LADDER = [48, 74, 96, 120]


def make(gamma=0.4, delta=1, ladder=LADDER, b_sat=0.9):
    return SpatialOracle(148, 148, ladder, b_sat, gamma, delta)


# ------------------------------------------------------------------ oracle pins --
def test_inactive_downstream_gets_the_aggressive_cap_and_active_never_exceeds_s_cap():
    o = make()
    for b in (0.0, 0.5, 5.0):
        assert o.update(False, b) == (148, 0)                      # Eq. 1, A = 0
    rng = np.random.default_rng(0)
    for _ in range(500):
        s, d = o.update(True, float(rng.uniform(0, 3)))
        assert s in LADDER and s <= 120 and s + d == 148           # bounded ladder, complementary headroom


def test_pressure_extremes_map_to_the_ends_of_the_ladder():
    lo, hi = make(gamma=1.0), make(gamma=1.0)
    assert lo.update(True, 0.0)[0] == 48                           # rho = 0 -> S_min
    assert hi.update(True, 0.9)[0] == 120                          # rho = 1 -> S_cap
    assert make(gamma=1.0).update(True, 50.0)[0] == 120            # clamped above saturation


def test_snap_takes_the_nearest_level_and_the_lower_one_on_a_tie():
    o = make()
    assert o.snap(48.0) == 48 and o.snap(60.9) == 48 and o.snap(61.1) == 74
    assert o.snap(61.0) == 48                                      # midpoint of 48 and 74
    assert o.snap(85.0) == 74                                      # midpoint of 74 and 96
    assert o.snap(1000.0) == 120 and o.snap(-5.0) == 48
    # gamma = 1: the cap is snap(S_min + rho (S_cap - S_min)), written out by hand for rho = 1/2: 84 -> 74
    assert make(gamma=1.0).update(True, 0.45)[0] == 74


def test_cap_is_monotone_in_the_pressure():
    caps = [make(gamma=1.0, delta=0).update(True, b)[0] for b in np.linspace(0, 1.2, 121)]
    assert all(x <= y for x, y in zip(caps, caps[1:])) and caps[0] == 48 and caps[-1] == 120


def test_ewma_closed_forms():
    o = make(gamma=0.4)
    o.update(True, 0.7)
    assert o.bhat == 0.7                                           # first sample initialises
    for _ in range(200):
        o.update(True, 0.7)
    assert abs(o.bhat - 0.7) < 1e-15                               # constant input is a fixed point
    # step response from 0 to 1 after k samples: 1 - (1 - gamma)^k
    o = make(gamma=0.4)
    o.update(False, 0.0)
    for k in range(1, 30):
        o.update(False, 1.0)
        assert abs(o.bhat - (1.0 - 0.6 ** k)) < 1e-12


def test_hysteresis_holds_the_cap_until_the_level_moves_far_enough():
    # ladder spacing 22..26; with delta_step = 30 a move by one level is ignored, by two levels it is taken
    o = make(gamma=1.0, delta=30)
    assert o.update(True, 0.0)[0] == 48                            # from 148: far enough
    assert o.update(True, 0.33)[0] == 48                           # s* = 74: 26 < 30, kept
    assert o.update(True, 0.62)[0] == 96                           # s* = 96: 48 >= 30, applied
    assert o.update(True, 0.33)[0] == 96                           # s* = 74: 22 < 30, kept
    assert o.update(False, 0.33)[0] == 148                         # inactive: applied at once
    assert o.update(True, 0.33)[0] == 74


def test_active_downstream_never_keeps_the_aggressive_cap_whatever_the_hysteresis():
    """Eq. 1 / Sec. 4.3: S_cap < S_aggr bounds the cap of every co-running step.  The case a hysteresis taken
    literally gets wrong: coming from the inactive case at 148 with maximum pressure, s* = 120 lies only 28 SMs
    away, less than delta_step = 30 -- the cap must still drop to 120 at once (and the downstream stage must be
    left with SMs)."""
    o = make(gamma=1.0, delta=30)
    assert o.update(False, 0.9) == (148, 0)
    assert o.update(True, 0.9) == (120, 28)
    rng = np.random.default_rng(11)
    for trial in range(60):
        n = int(rng.integers(1, 7))
        ladder = sorted(rng.choice(np.arange(8, 140), size=n, replace=False).tolist())
        s_aggr = int(rng.integers(ladder[-1] + 1, 149))
        o = SpatialOracle(148, s_aggr, ladder, float(rng.uniform(0.2, 2.0)), float(rng.uniform(0.05, 1.0)),
                          int(rng.integers(0, 60)))
        active = False
        for _ in range(300):
            if rng.uniform() < 0.15:
                active = not active
            s, d = o.update(active, float(rng.uniform(0, 2.5)))
            if active:
                assert s in ladder and s <= ladder[-1] < s_aggr and d == 148 - s and d > 0, (trial, s)
            else:
                assert s == s_aggr


def test_derive_cap_smallest_near_best_budget_below_full_allocation():
    # decode latency saturates at 80 SMs and gets worse at full allocation (the shape of the paper's Fig. 4)
    budgets = [16, 32, 48, 64, 80, 96, 120, 142]
    lat = [40.0, 22.0, 16.0, 13.2, 12.9, 12.8, 12.85, 14.0]
    assert derive_cap(budgets, lat, 142, 0.05) == 64               # 13.2 <= 12.8 * 1.05
    assert derive_cap(budgets, lat, 142, 0.0) == 96
    assert derive_cap(budgets, lat, 142, 10.0) == 16
    assert derive_cap([148, 74], [1.0, 5.0], 148, 0.05) == 74      # only one candidate below the total


# ------------------------------------------------------------- library vs oracle --
def test_library_controller_matches_the_oracle_decision_by_decision():
    from paper_2608_01785_b200 import binding as B
    rng = np.random.default_rng(7)
    for trial in range(40):
        n = int(rng.integers(1, 9))
        ladder = sorted(rng.choice(np.arange(1, 140), size=n, replace=False).tolist())
        s_aggr = int(rng.integers(ladder[-1] + 1, 149))
        gamma = float(rng.uniform(0.05, 1.0))
        b_sat = float(rng.uniform(0.2, 2.0))
        delta = int(rng.integers(0, 40))
        orc = SpatialOracle(148, s_aggr, ladder, b_sat, gamma, delta)
        ctl = B.SpatialController(148, s_aggr, ladder, b_sat, gamma, delta)
        assert ctl.state() == (0.0, s_aggr)
        active = False
        for step in range(400):
            if rng.uniform() < 0.1:
                active = not active
            b = float(rng.choice([rng.uniform(0, 2.5), 0.0, b_sat, b_sat / 2]))
            assert ctl.update(active, b) == orc.update(active, b), (trial, step)
            bhat, s = ctl.state()
            assert bhat == orc.bhat and s == orc.s_shared          # same double arithmetic, same order
        ctl.close()


def test_library_controller_argument_errors():
    from paper_2608_01785_b200 import binding as B
    bad = [dict(ladder=[]), dict(ladder=[74, 48]), dict(ladder=[48, 48]), dict(ladder=[0, 48]), dict(ladder=[48, 148]),
           dict(s_aggr=120), dict(s_aggr=149), dict(b_sat=0.0), dict(b_sat=float("nan")), dict(gamma=0.0),
           dict(gamma=1.5), dict(delta_step=-1)]
    for kw in bad:
        args = dict(s_total=148, s_aggr=148, ladder=LADDER, b_sat=0.9, gamma=0.4, delta_step=1)
        args.update(kw)
        with pytest.raises(B.HsError) as e:
            B.SpatialController(**args)
        assert e.value.status == B.HS_ERR_INVALID_ARG, kw
    ctl = B.SpatialController(148, 148, LADDER, 0.9, 0.4, 1)
    ctl.update(True, 0.5)
    before = ctl.state()
    for b in (-0.1, float("inf"), float("nan")):
        with pytest.raises(B.HsError):
            ctl.update(True, b)
    assert ctl.state() == before                                   # a refused sample changes nothing
    ctl.close()


def test_library_derive_cap_matches_the_oracle():
    from paper_2608_01785_b200 import binding as B
    rng = np.random.default_rng(3)
    for _ in range(200):
        n = int(rng.integers(2, 10))
        budgets = rng.choice(np.arange(1, 149), size=n, replace=False).tolist()
        if min(budgets) == 148:
            continue
        lat = rng.uniform(1.0, 20.0, size=n).tolist()
        tol = float(rng.choice([0.0, 0.05, 0.2, 3.0]))
        assert B.hs_spatial_derive_cap(budgets, lat, 148, tol) == derive_cap(budgets, lat, 148, tol)
    with pytest.raises(B.HsError):
        B.hs_spatial_derive_cap([148], [1.0], 148, 0.05)           # nothing below the full allocation
    with pytest.raises(B.HsError):
        B.hs_spatial_derive_cap([74, 74], [1.0, 2.0], 148, 0.05)   # budgets must be distinct
