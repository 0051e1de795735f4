"""Co-run harness: the shared stage and a downstream stage on two CUDA streams of one GPU with
complementary SM budgets (the paper's spatial sharing: s_down = S_tot - s_shared, Sec. 4.3), measured
against each stage running alone at the same budget.  Only launches and timing live here."""
from __future__ import annotations

import threading
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
    Each stage is driven by a host thread of its own (as two serving processes would), with at most two steps
    queued ahead of the device, so that neither stream waits for the other's launches: one thread feeding
    both streams is paced by the stream with more launches once the driver's launch queue fills.  Stage B
    keeps stepping until stage A's last step has completed; the at most two B steps that finish after that
    are part of its average (negligible at the default step count)."""
    budget_b = stage_a.sm_count - budget_a
    dev = stage_a.device
    sa, sb = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    solo_a = _time_solo(stage_a, batch_a, budget_a, steps, sa)
    solo_b = _time_solo(stage_b, batch_b, budget_b, steps, sb)
    ea0, ea1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    eb0, eb1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    go = threading.Barrier(2)
    stop = threading.Event()
    count = {"b": 0}
    errors = []

    def drive(stage, batch, budget, stream, n_steps, e_first, e_last, key):
        try:
            torch.cuda.set_device(dev)
            go.wait(timeout=60)
            e_first.record(stream)
            done = []
            i = 0
            while (i < n_steps) if n_steps else not stop.is_set():
                if len(done) >= 2:
                    done.pop(0).synchronize()
                stage.step(batch, budget, stream)
                ev = torch.cuda.Event()
                ev.record(stream)
                done.append(ev)
                i += 1
            e_last.record(stream)
            e_last.synchronize()
            if key:
                count[key] = i
        except Exception as exc:        # surfaced by the caller
            errors.append(exc)
        finally:
            if not key:
                stop.set()

    torch.cuda.synchronize()
    ta = threading.Thread(target=drive, args=(stage_a, batch_a, budget_a, sa, steps, ea0, ea1, None))
    tb = threading.Thread(target=drive, args=(stage_b, batch_b, budget_b, sb, 0, eb0, eb1, "b"))
    ta.start()
    tb.start()
    ta.join()
    tb.join()
    torch.cuda.synchronize()
    if errors:
        raise errors[0]
    n_b = max(count["b"], 1)
    return {"budget_a": budget_a, "budget_b": budget_b, "solo_a_ms": solo_a, "solo_b_ms": solo_b,
            "corun_a_ms": ea0.elapsed_time(ea1) / steps, "corun_b_ms": eb0.elapsed_time(eb1) / n_b,
            "b_steps_per_a_step": round(n_b / steps, 2)}
