"""The temporal scheduler's view (Sec. 4.1-4.2, Algorithm 1 steps 1-2): oracle pins, then library vs oracle."""
import numpy as np
import pytest

from oracle.temporal import DECODE, LONG, PREFILL, SHORT, Req, TemporalOracle


def R(rid, path, stage=PREFILL, deadline=1e9, remaining=1.0):
    return Req(rid, path, stage, deadline, remaining)


# ------------------------------------------------------------------ oracle pins --
def test_rotation_pattern_is_n_short_steps_then_m_long_steps():
    o = TemporalOracle(n_min=2, n_max=8, m=2)
    reqs = [R(0, SHORT), R(1, LONG)]                       # nobody protected: N stays at N_min = 2
    phases = [o.step(0.0, reqs, 0)[1] for _ in range(12)]
    assert phases == [SHORT, SHORT, LONG, LONG] * 3        # k mod (N + M) < N
    # in a short phase the ordinary long-path prefill is hidden, in a long phase the short-path one
    o = TemporalOracle()
    assert o.step(0.0, reqs, 0)[0] == [True, False]
    o.step(0.0, reqs, 0)
    assert o.step(0.0, reqs, 0)[0] == [False, True]


def test_decode_and_protected_requests_stay_visible_in_every_phase():
    o = TemporalOracle(u_guard=1.5)
    reqs = [R(0, LONG, DECODE), R(1, LONG, PREFILL, deadline=1.2, remaining=1.0),      # u = 1.2 < 1.5: protected
            R(2, LONG, PREFILL, deadline=10.0, remaining=1.0), R(3, SHORT, DECODE)]
    for _ in range(8):
        vis, phase, _ = o.step(0.0, reqs, 0)
        assert vis[0] and vis[1] and vis[3]
        assert vis[2] == (phase == LONG)


def test_slack_ratio_and_guard_band():
    o = TemporalOracle(u_guard=1.5)
    assert o.protected(R(0, SHORT, deadline=14.9, remaining=10.0), 0.0)          # u = 1.49
    assert not o.protected(R(0, SHORT, deadline=15.0, remaining=10.0), 0.0)      # u = 1.5 is not below the guard
    assert o.protected(R(0, SHORT, deadline=15.0, remaining=10.0), 0.5)          # time passes: u = 1.45
    assert o.protected(R(0, SHORT, deadline=1.0, remaining=10.0), 2.0)           # past its deadline
    assert not o.protected(R(0, SHORT, deadline=1.0, remaining=0.0), 0.0)        # nothing left to do, deadline ahead


def test_adaptive_n_follows_the_protected_fraction_of_waiting_short_requests():
    def n_for(n_prot, n_ok):
        o = TemporalOracle(n_min=2, n_max=8, m=2, u_guard=1.5)
        reqs = [R(i, SHORT, deadline=1.0, remaining=1.0) for i in range(n_prot)] + \
               [R(100 + i, SHORT, deadline=100.0, remaining=1.0) for i in range(n_ok)] + [R(999, LONG)]
        return o.step(0.0, reqs, 0)[2]
    assert n_for(0, 5) == 2 and n_for(5, 0) == 8                 # f = 0 -> N_min, f = 1 -> N_max
    assert n_for(1, 1) == 5                                      # f = 1/2 -> 2 + 3
    assert n_for(1, 3) == 4                                      # f = 1/4 -> 3.5 -> rounds up to 4
    assert n_for(0, 0) == 2                                      # no waiting short-path prefill
    # long-path share at maximum pressure: M / (N_max + M) = 20 % of the steps
    o = TemporalOracle()
    reqs = [R(0, SHORT, deadline=0.5, remaining=1.0), R(1, LONG)]
    phases = [o.step(0.0, reqs, 0)[1] for _ in range(100)]
    assert phases.count(LONG) == 20
    # N changes only when a cycle starts
    o = TemporalOracle()
    calm, tense = [R(0, SHORT, deadline=100.0)], [R(0, SHORT, deadline=0.1)]
    seq = [o.step(0.0, calm, 0)[2]] + [o.step(0.0, tense, 0)[2] for _ in range(4)]
    assert seq == [2, 2, 2, 2, 8]                                # cycle of 2 + 2 steps, then the new N


def test_long_path_cap_keeps_the_earliest_deadlines():
    o = TemporalOracle(n_min=2, m=2, long_cap=3)
    o.step(0.0, [], 0)
    o.step(0.0, [], 0)                                           # next step is a long-path phase
    reqs = [R(0, LONG, deadline=50.0), R(1, LONG, deadline=20.0), R(2, LONG, deadline=30.0),
            R(3, LONG, deadline=20.0), R(4, LONG, deadline=1.0, remaining=1.0),      # protected: exempt
            R(5, LONG, DECODE), R(6, SHORT)]
    vis, phase, _ = o.step(0.0, reqs, 1)                         # one slot already taken: room for two
    assert phase == LONG
    assert vis == [False, True, False, True, True, True, False]  # deadlines 20 (ids 1, 3) win; 4 and 5 exempt
    o2 = TemporalOracle(n_min=2, m=2, long_cap=3)
    o2.step(0.0, [], 0); o2.step(0.0, [], 0)
    assert o2.step(0.0, reqs, 5)[0] == [False, False, False, False, True, True, False]   # no room at all


# ------------------------------------------------------------- library vs oracle --
def test_library_view_matches_the_oracle_step_by_step():
    from paper_2608_01785_b200 import binding as B
    rng = np.random.default_rng(11)
    for trial in range(30):
        n_min = int(rng.integers(1, 4))
        n_max = int(rng.integers(n_min, 10))
        m = int(rng.integers(1, 4))
        guard = float(rng.uniform(0.8, 3.0))
        cap = int(rng.integers(0, 6))
        orc = TemporalOracle(n_min, n_max, m, guard, cap)
        lib = B.TemporalView(n_min, n_max, m, guard, cap)
        now = 0.0
        for step in range(200):
            now += float(rng.uniform(0.0, 0.05))
            n = int(rng.integers(0, 14))
            reqs = [Req(int(rng.integers(0, 1000)), int(rng.integers(0, 2)), int(rng.integers(0, 2)),
                        now + float(rng.choice([rng.uniform(-0.2, 3.0), 0.5, 1.0])),
                        float(rng.choice([rng.uniform(0.0, 2.0), 0.0, 0.5]))) for _ in range(n)]
            admitted = int(rng.integers(0, 7))
            want = orc.step(now, reqs, admitted)
            got = lib.step(now, [(r.rid, r.path, r.stage, r.deadline, r.remaining) for r in reqs], admitted)
            assert got == (want[0], want[1], want[2]), (trial, step)
        lib.close()


def test_library_view_argument_errors():
    from paper_2608_01785_b200 import binding as B
    for kw in (dict(n_min=0), dict(n_min=5, n_max=4), dict(n_max=65), dict(m=0), dict(u_guard=0.0), dict(long_cap=-1)):
        with pytest.raises(B.HsError):
            B.TemporalView(**kw)
    v = B.TemporalView()
    assert v.step(0.0, [], 0) == ([], SHORT, 2)
    with pytest.raises(B.HsError):
        v.step(0.0, [(1, 2, 0, 1.0, 1.0)], 0)                   # path outside {0, 1}
    with pytest.raises(B.HsError):
        v.step(0.0, [(1, 0, 0, float("nan"), 1.0)], 0)
    assert v.step(0.0, [], 0)[1] == SHORT                        # the refused steps did not advance the rotation
    assert v.step(0.0, [], 0)[1] == LONG
    v.close()


def _paper_constants():
    import os
    out = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "paper_scheduler_constants.txt")):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


def test_defaults_and_long_path_share_match_the_values_the_paper_prints():
    """tests/golden/paper_scheduler_constants.txt holds what the paper states (Sec. 4.2, Sec. 6.4)."""
    c = _paper_constants()
    o = TemporalOracle()
    assert (o.n_min, o.n_max, o.m) == (c["rotation_n_min"], c["rotation_n_max"], c["rotation_m"])
    reqs = [R(0, SHORT, deadline=0.5, remaining=1.0), R(1, LONG)]       # every waiting short-path request protected
    phases = [o.step(0.0, reqs, 0)[1] for _ in range(1000)]
    assert abs(phases.count(LONG) / 1000 - c["long_share_at_max_pressure"]) < 1e-12
    from paper_2608_01785_b200.replay import ReplayConfig
    assert ReplayConfig().gamma == c["ewma_gamma"]
