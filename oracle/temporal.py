"""Oracle of the temporal scheduler's view (TEST INFRASTRUCTURE ONLY): which requests the base scheduler may
see in one scheduling step -- shared-stage path rotation, slack guard, adaptive rotation ratio and long-path
admission cap of the paper (Sec. 4.1 "Remaining-slack ratio", Sec. 4.2, Algorithm 1 steps 1-2).

A request is (id, path, stage, deadline, remaining): path 0 = short (ends after the shared stage), 1 = long
(activates a downstream stage); stage 0 = waiting for / in prefill, 1 = decode continuation.

    u_i      = (d_i - t) / rhat_i                      protected_i = u_i < u_guard
    phase(k) = short while the position in the cycle is < N, long for the following M steps
    N        = round(N_min + f (N_max - N_min)),  f = protected fraction of the waiting short-path prefills
    visible  = decode continuations, protected requests, and prefills whose path is the phase's;
               of the visible ordinary long-path prefills only the long_cap - long_admitted with the earliest
               deadlines stay visible

Readings where the paper is silent: N is re-evaluated when a cycle starts (the phase pattern of a running
cycle is not changed under it); rounding is to nearest, halves up; with no waiting short-path prefill f = 0;
ties of deadlines go to the lower id; rhat <= 0 counts as protected only if the deadline has passed or is now.

Parity status: no worked example in the paper (paper-level parity unpinned); pinned by hand-worked cases and
invariants in tests/test_temporal.py.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Sequence, Tuple

SHORT, LONG = 0, 1
PREFILL, DECODE = 0, 1


@dataclass
class Req:
    rid: int
    path: int
    stage: int
    deadline: float
    remaining: float     # rhat: estimated time the request still needs to its first response


class TemporalOracle:
    def __init__(self, n_min: int = 2, n_max: int = 8, m: int = 2, u_guard: float = 1.5, long_cap: int = 4):
        self.n_min, self.n_max, self.m, self.u_guard, self.long_cap = n_min, n_max, m, u_guard, long_cap
        self.n = n_min
        self.pos = 0         # position inside the current cycle of n + m steps

    def protected(self, r: Req, now: float) -> bool:
        slack = r.deadline - now
        if r.remaining <= 0.0:
            return slack <= 0.0
        return slack / r.remaining < self.u_guard

    def step(self, now: float, reqs: Sequence[Req], long_admitted: int) -> Tuple[List[bool], int, int]:
        """Returns (visible flag per request, phase of this step, N in force)."""
        prot = [self.protected(r, now) for r in reqs]
        if self.pos == 0:                                   # a cycle starts: adapt the short-path share
            short_wait = [p for r, p in zip(reqs, prot) if r.path == SHORT and r.stage == PREFILL]
            f = sum(short_wait) / len(short_wait) if short_wait else 0.0
            self.n = int(math.floor(self.n_min + f * (self.n_max - self.n_min) + 0.5))
        phase = SHORT if self.pos < self.n else LONG
        self.pos = (self.pos + 1) % (self.n + self.m)
        visible = [r.stage == DECODE or p or r.path == phase for r, p in zip(reqs, prot)]
        # long-path admission cap on the ordinary (unprotected) long-path prefills that are still visible
        cand = [i for i, (r, p) in enumerate(zip(reqs, prot))
                if visible[i] and r.stage == PREFILL and r.path == LONG and not p]
        room = max(0, self.long_cap - long_admitted)
        cand.sort(key=lambda i: (reqs[i].deadline, reqs[i].rid))
        for i in cand[room:]:
            visible[i] = False
        return visible, phase, self.n
