"""Co-run harness: the shared stage and a downstream stage on two CUDA streams of one GPU with
complementary SM budgets (the paper's spatial sharing: s_down = S_tot - s_shared, Sec. 4.3), measured
against each stage running alone at the same budget.  Only launches and timing live here."""
from __future__ import annotations

from typing import Dict

import torch

from .stage import Stage


def _time_solo(stage: Stage, batch, budget: int, steps: int, stream: torch.cuda.Stream) -> float:
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    for _ in range(3):
        stage.step(batch, budget, stream)
    e0.record(stream)
    for _ in range(steps):
        stage.step(batch, budget, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def corun(stage_a: Stage, batch_a, stage_b: Stage, batch_b, budget_a: int, steps: int = 10) -> Dict[str, float]:
    """Runs `steps` steps of stage A at budget_a while stage B runs back to back at S_tot - budget_a.

    Returns per-step latencies in ms: each stage alone at its budget, and both while they overlap.
    Stage B is given enough steps to stay busy for as long as stage A runs."""
    budget_b = stage_a.sm_count - budget_a
    sa, sb = torch.cuda.Stream(device=stage_a.device), torch.cuda.Stream(device=stage_a.device)
    solo_a = _time_solo(stage_a, batch_a, budget_a, steps, sa)
    solo_b = _time_solo(stage_b, batch_b, budget_b, steps, sb)
    ratio = max(1, int(round(solo_a / solo_b)))
    ea0, ea1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    eb0, eb1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    go = torch.cuda.Event()
    torch.cuda.synchronize()
    go.record()
    sa.wait_event(go)
    sb.wait_event(go)
    ea0.record(sa)
    eb0.record(sb)
    n_b = 0
    for _ in range(steps):
        stage_a.step(batch_a, budget_a, sa)
        for _ in range(ratio):
            stage_b.step(batch_b, budget_b, sb)
            n_b += 1
    ea1.record(sa)
    eb1.record(sb)
    torch.cuda.synchronize()
    return {"budget_a": budget_a, "budget_b": budget_b, "solo_a_ms": solo_a, "solo_b_ms": solo_b,
            "corun_a_ms": ea0.elapsed_time(ea1) / steps, "corun_b_ms": eb0.elapsed_time(eb1) / n_b,
            "b_steps_per_a_step": ratio}
