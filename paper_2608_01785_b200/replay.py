"""Replay of a downstream-heavy request trace on the two stages (backbone + talker) of one GPU.

Each scheduler tick issues one backbone step (every sequence in its decode phase, at most `max_decode`, plus
one first-come-first-served prefill chunk of at most `max_prefill_chunk` tokens) and, when downstream work
exists, one talker step (at most `max_talker` sequences) on a second stream with the complementary SM
budget -- the co-running regime whose SM split the paper's spatial controller chooses per step (Sec. 4.3,
Algorithm 1 steps 3-4).  The per-tick backbone budget comes from one of two policies: "seeded" (all SMs when
the talker is idle, otherwise a uniform draw from the ladder: it visits every budget equally often, which is
what the latency-by-budget tables want) or "controller" (the library's spatial controller, Eq. 1 of the
paper, driven by a measured pressure sample per tick: the bytes the two steps of the previous tick had to
read -- weights once per step, the KV pages of every sequence -- divided by the tick's duration and by the
GPU's measured copy bandwidth).  Time is virtual: the clock advances by the
measured latency of each tick and idle gaps are skipped, so a long trace replays in GPU time only.

With `image_stage = "dit"` the image class's downstream stage is a third stage, the conditioned denoising
stage without a causal mask (workload c6_dit): an image runs `dit_steps` steps over its `dit_tokens` latent
tokens, at most `max_dit` images per step, each step behind the talker's on the downstream stream.

The engine is pluggable: `GpuEngine` drives real stages through the C ABI; `ModelEngine` is a latency
model used by the CPU tests of the scheduling logic (it runs the same page accounting on host-only
stages, so allocator pressure is exercised without a GPU).
"""
from __future__ import annotations

import argparse
import json
import statistics
from collections import deque
from dataclasses import dataclass, field
from typing import Deque, Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import binding as B
from . import workloads as wl


@dataclass
class ReplayConfig:
    max_decode: int = 64
    max_prefill_chunk: int = 2048
    max_talker: int = 16
    talker_ctx0: int = 128          # conditioning tokens a talker sequence starts from
    ladder: Tuple[int, ...] = (120, 96, 74, 48)
    policy_seed: int = 5
    policy: str = "seeded"          # "seeded" | "controller" | "horizon" (temporal view + spatial controller)
    hbm_gbs: float = 6547.2         # measured copy bandwidth: normalises the controller's pressure samples
    b_sat: float = 0.5              # pressure (fraction of hbm_gbs) at which the cap reaches the top of the ladder
    gamma: float = 0.4              # weight of the newest pressure sample (the value of the paper's Fig. 10)
    delta_step: int = 20            # smallest change of the cap that is applied while co-running (SMs)
    # first-response deadlines per class (ms after arrival): text = first backbone token, speech / image = first
    # downstream step.  Stand-ins for the paper's "solo p95 x multiplier" table (Sec. 4.1)
    slo_ms: Tuple[Tuple[str, float], ...] = (("text", 120.0), ("speech", 1500.0), ("image", 1500.0))
    u_guard: float = 1.5            # slack-ratio guard band
    long_cap: int = 24              # most ordinary long-path requests holding backbone slots
    est_fixed_ms: float = 8.0       # coarse remaining-time estimate: fixed part (one tick) ...
    est_per_token_ms: float = 0.014 # ... + per prompt token still to prefill ...
    est_down_ms: float = 8.0        # ... + one more tick for the first downstream step of a long-path request
    # downstream stage of the image class: "talker" (talker-shaped steps, the stand-in) or "dit": a conditioned
    # denoising stage without a causal mask that runs dit_steps steps over dit_tokens latent tokens per image,
    # at most max_dit images per step, after the talker's step on the downstream stream
    image_stage: str = "talker"
    dit_steps: int = 20
    dit_tokens: int = 256
    max_dit: int = 4


@dataclass
class _Seq:
    req: wl.Request
    prefilled: int = 0              # prompt tokens already in the cache
    decoded: int = 0                # backbone tokens generated
    talker_done: int = 0
    dit_done: int = 0
    t_first: Optional[float] = None       # first backbone token (end of the tick that finished prefill)
    t_first_down: Optional[float] = None  # first downstream token
    t_done: Optional[float] = None


class Engine:
    """Runs one tick; returns (backbone ms, talker ms, denoising-stage ms), None where a stage had no batch."""
    sm_count = 148
    dims_c = None

    def tick(self, a_batch, b_batch, budget_a: int, c_batch=None):
        raise NotImplementedError

    def alloc(self, which: str, seq_id: int, total: int) -> None:
        raise NotImplementedError

    def free(self, which: str, seq_id: int) -> None:
        raise NotImplementedError


class ModelEngine(Engine):
    """Latency model + real page accounting on host-only stages (no GPU)."""

    def __init__(self, dims_a, dims_b, pages_a: int, pages_b: int, mpps_a: int, mpps_b: int, dims_c=None,
                 pages_c: int = 0, mpps_c: int = 0):
        self.dims_a, self.dims_b, self.dims_c = dims_a, dims_b, dims_c
        self.h = {}
        stages = [("a", dims_a, pages_a, mpps_a), ("b", dims_b, pages_b, mpps_b)]
        if dims_c is not None:
            stages.append(("c", dims_c, pages_c, mpps_c))
        for name, dims, pages, mpps in stages:
            cfg = B.make_config(dims, pages, 4096, 128, mpps, mpps * 16, device=-1)
            self.h[name] = (B.hs_stage_create(cfg, None, 0, 0), mpps)

    def alloc(self, which, seq_id, total):
        h, mpps = self.h[which]
        B.hs_kv_alloc(h, seq_id, total, mpps)

    def free(self, which, seq_id):
        B.hs_kv_free(self.h[which][0], seq_id)

    def free_pages(self, which):
        return B.hs_kv_free_pages(self.h[which][0])

    def tick(self, a_batch, b_batch, budget_a, c_batch=None):
        la = lb = lc = None
        if a_batch:
            toks = sum(q for _, q, _ in a_batch)
            la = (2.0 + 0.012 * toks) * self.sm_count / budget_a
        if b_batch:
            lb = 1.2 * self.sm_count / max(self.sm_count - budget_a, 1) ** 0.3 / 4.0
        if c_batch:
            lc = (0.6 + 0.0006 * sum(q for _, q, _ in c_batch)) * (self.sm_count / max(self.sm_count - budget_a, 28)) ** 0.5
        return la, lb, lc

    def close(self):
        for h, _ in self.h.values():
            B.hs_stage_destroy(h)


class GpuEngine(Engine):
    """Two real stages on one GPU, stepped on two streams with complementary budgets."""

    def __init__(self, dims_a, dims_b, pages_a: int, pages_b: int, mpps_a: int, mpps_b: int, cfg: ReplayConfig,
                 seed: int = 4, device: int = 0, dims_c=None):
        import torch
        from .stage import Stage
        self.torch = torch
        self.dims_a, self.dims_b = dims_a, dims_b
        dev = torch.device("cuda", device)
        max_tok_a = cfg.max_decode + cfg.max_prefill_chunk
        self.sa = Stage(dims_a, wl.make_weights(dims_a, seed, dev), pages_a, max_tok_a, cfg.max_decode + 1, mpps_a,
                        mpps_a * 16, device)
        self.sb = Stage(dims_b, wl.make_weights(dims_b, seed + 1, dev), pages_b, cfg.max_talker, cfg.max_talker, mpps_b,
                        mpps_b * 16, device)
        self.sm_count = self.sa.sm_count
        self.xa = wl.make_x(max_tok_a, dims_a.d_model, seed, dev)
        self.xb = wl.make_x(cfg.max_talker, dims_b.d_model, seed + 1, dev)
        self.ya = torch.empty(max_tok_a, dims_a.d_model, dtype=torch.float32, device=dev)
        self.yb = torch.empty(cfg.max_talker, dims_b.d_model, dtype=torch.float32, device=dev)
        self.stream_a, self.stream_b = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        self.tables = {"a": {}, "b": {}, "c": {}}
        self.dims_c, self.sc = dims_c, None
        if dims_c is not None:      # the denoising stage: no causal mask, conditioned, an image's pages live for its steps
            mpps_c = -(-cfg.dit_tokens // 16)
            max_tok_c = cfg.max_dit * cfg.dit_tokens
            self.sc = Stage(dims_c, wl.make_weights(dims_c, seed + 2, dev), cfg.max_dit * mpps_c, max_tok_c, cfg.max_dit,
                            mpps_c, cfg.dit_tokens, device, B.HS_FLAG_BIDIRECTIONAL)
            self.sc.set_modulation(wl.make_modulation(dims_c, cfg.max_dit, seed + 2, dev))
            self.xc = wl.make_x(max_tok_c, dims_c.d_model, seed + 2, dev)
            self.yc = torch.empty(max_tok_c, dims_c.d_model, dtype=torch.float32, device=dev)

    def _stage(self, which):
        return {"a": self.sa, "b": self.sb, "c": self.sc}[which]

    def alloc(self, which, seq_id, total):
        self.tables[which][seq_id] = self._stage(which).kv_alloc(seq_id, total)

    def free(self, which, seq_id):
        self._stage(which).kv_free(seq_id)
        del self.tables[which][seq_id]

    def free_pages(self, which):
        return B.hs_kv_free_pages(self._stage(which).handle)

    def _launch(self, which, batch, budget, stream, x, y):
        st = self._stage(which)
        bt = st.block_table_array([self.tables[which][sid] for sid, _, _ in batch])
        n = sum(q for _, q, _ in batch)
        b = st.make_batch([q for _, q, _ in batch], [c for _, _, c in batch], bt, x[:n], y[:n])
        e0, e1 = self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        st.step(b, budget, stream)
        e1.record(stream)
        return e0, e1, b

    def tick(self, a_batch, b_batch, budget_a, c_batch=None):
        ev = []
        down = self.sm_count - budget_a if a_batch else self.sm_count
        if a_batch:
            ev.append(("a",) + self._launch("a", a_batch, budget_a, self.stream_a, self.xa, self.ya))
        if b_batch:
            ev.append(("b",) + self._launch("b", b_batch, down, self.stream_b, self.xb, self.yb))
        if c_batch:                 # behind the talker's step on the downstream stream, same SM share
            ev.append(("c",) + self._launch("c", c_batch, down, self.stream_b, self.xc, self.yc))
        self.torch.cuda.synchronize()
        out = {"a": None, "b": None, "c": None}
        for which, e0, e1, _ in ev:
            out[which] = e0.elapsed_time(e1)
        assert self.sa.status() == 0 and self.sb.status() == 0 and (self.sc is None or self.sc.status() == 0)
        return out["a"], out["b"], out["c"]

    def close(self):
        self.sa.close()
        self.sb.close()
        if self.sc is not None:
            self.sc.close()


def step_bytes(dims, batch) -> float:
    """Bytes one step of a stage has to read: its weights once, and the cached K/V of every sequence."""
    if not batch:
        return 0.0
    kv = sum(ctx + q for _, q, ctx in batch) * 2 * dims.kv_dim * 2 * dims.n_layers
    return float(dims.params_per_layer() * dims.n_layers * 2 + kv)


def replay(trace: Sequence[wl.Request], engine: Engine, cfg: ReplayConfig = ReplayConfig()) -> Dict:
    """Runs the whole trace; returns aggregate metrics (virtual seconds)."""
    rng = np.random.Generator(np.random.PCG64(cfg.policy_seed))
    ctl = None
    if cfg.policy == "controller":
        ctl = B.SpatialController(engine.sm_count, engine.sm_count, sorted(cfg.ladder), cfg.b_sat, cfg.gamma,
                                  cfg.delta_step)
    pressure = 0.0                  # sample of the previous tick
    pressures: List[float] = []
    cap_changes = 0
    prev_budget = None
    waiting: Deque[_Seq] = deque()
    prefilling: Optional[_Seq] = None
    decoding: List[_Seq] = []
    talker_wait: Deque[_Seq] = deque()
    talking: List[_Seq] = []
    use_dit = cfg.image_stage == "dit" and engine.dims_c is not None
    dit_wait: Deque[_Seq] = deque()
    denoising: List[_Seq] = []
    dit_lat: List[float] = []
    dit_tokens = 0
    done: List[_Seq] = []
    t = 0.0
    nxt = 0
    ticks_by_budget: Dict[int, List[float]] = {}
    talker_lat: List[float] = []
    backbone_tokens = talker_tokens = 0
    busy_s = 0.0

    def admit(now):
        nonlocal nxt
        while nxt < len(trace) and trace[nxt].arrival_s <= now:
            waiting.append(_Seq(trace[nxt]))
            nxt += 1

    slo = dict(cfg.slo_ms)
    view = B.TemporalView(2, 8, 2, cfg.u_guard, cfg.long_cap) if cfg.policy == "horizon" else None
    if view is not None and ctl is None:
        ctl = B.SpatialController(engine.sm_count, engine.sm_count, sorted(cfg.ladder), cfg.b_sat, cfg.gamma,
                                  cfg.delta_step)

    def is_long(s):
        return s.req.talker_out > 0

    def down_finished(s):
        if use_dit and s.req.out_class == "image":
            return s.dit_done >= cfg.dit_steps
        return s.req.talker_out == 0 or s.talker_done >= s.req.talker_out

    def deadline(s):
        return s.req.arrival_s + slo[s.req.out_class] * 1e-3

    def remaining(s):
        est = cfg.est_fixed_ms + cfg.est_per_token_ms * (s.req.prompt_len - s.prefilled)
        return (est + (cfg.est_down_ms if is_long(s) else 0.0)) * 1e-3

    def pick_next():
        """The base scheduler (first come, first served) on the temporal view of this step."""
        if view is None:
            return waiting.popleft()
        reqs = [(s.req.rid, int(is_long(s)), 0, deadline(s), remaining(s)) for s in waiting] + \
               [(s.req.rid, int(is_long(s)), 1, deadline(s), 0.0) for s in decoding]
        admitted = sum(1 for s in decoding if is_long(s))
        visible, _, _ = view.step(t, reqs, admitted)
        for i, s in enumerate(waiting):
            if visible[i]:
                del waiting[i]
                return s
        return None

    while len(done) < len(trace):
        admit(t)
        if prefilling is None and waiting and len(decoding) < cfg.max_decode:
            prefilling = pick_next()
        while talker_wait and len(talking) < cfg.max_talker:
            s = talker_wait.popleft()
            talking.append(s)
        while dit_wait and len(denoising) < cfg.max_dit:
            denoising.append(dit_wait.popleft())
        if prefilling is None and not decoding and not talking and not denoising:
            if waiting:
                continue                              # everything waiting was hidden in this phase: next step
            if nxt >= len(trace):
                break
            t = max(t, trace[nxt].arrival_s)          # idle: jump to the next arrival
            continue

        # ---- build the tick's batches: (seq id, new tokens, cached tokens) ----
        a_batch = []
        if prefilling is not None:
            n = min(cfg.max_prefill_chunk, prefilling.req.prompt_len - prefilling.prefilled)
            engine.alloc("a", prefilling.req.rid, prefilling.prefilled + n)
            a_batch.append((prefilling.req.rid, n, prefilling.prefilled))
        stepped = list(decoding)                       # sequences that decode one token in this tick
        for s in stepped:
            ctx = s.req.prompt_len + s.decoded
            engine.alloc("a", s.req.rid, ctx + 1)
            a_batch.append((s.req.rid, 1, ctx))
        b_batch = []
        for s in talking:
            ctx = cfg.talker_ctx0 + s.talker_done
            engine.alloc("b", s.req.rid, ctx + 1)
            b_batch.append((s.req.rid, 1, ctx))
        c_batch = []
        for s in denoising:                            # a denoising step sees the whole image, nothing is cached
            engine.alloc("c", s.req.rid, cfg.dit_tokens)
            c_batch.append((s.req.rid, cfg.dit_tokens, 0))
        down_active = bool(b_batch) or bool(c_batch)
        if ctl is not None:
            budget, _ = ctl.update(down_active, pressure)
        else:
            budget = engine.sm_count if not down_active else int(rng.choice(cfg.ladder))
        if prev_budget is not None and budget != prev_budget:
            cap_changes += 1
        prev_budget = budget
        lat_a, lat_b, lat_c = engine.tick(a_batch, b_batch, budget, c_batch)
        tick_ms = max(lat_a or 0.0, (lat_b or 0.0) + (lat_c or 0.0))     # the two downstream steps share a stream
        moved = step_bytes(engine.dims_a, a_batch) + step_bytes(engine.dims_b, b_batch)
        if c_batch:
            moved += step_bytes(engine.dims_c, c_batch)
        pressure = moved / (tick_ms * 1e-3) / (cfg.hbm_gbs * 1e9) if tick_ms > 0 else 0.0
        pressures.append(pressure)
        t += tick_ms * 1e-3
        busy_s += tick_ms * 1e-3
        if lat_a is not None:
            ticks_by_budget.setdefault(budget, []).append(lat_a)
            backbone_tokens += sum(q for _, q, _ in a_batch)
        if lat_b is not None:
            talker_lat.append(lat_b)
            talker_tokens += len(b_batch)
        if lat_c is not None:
            dit_lat.append(lat_c)
            dit_tokens += cfg.dit_tokens * len(c_batch)

        # ---- advance request state ----
        if prefilling is not None:
            prefilling.prefilled += a_batch[0][1]
            if prefilling.prefilled == prefilling.req.prompt_len:
                prefilling.t_first = t
                decoding.append(prefilling)
                if use_dit and prefilling.req.out_class == "image":
                    dit_wait.append(prefilling)
                elif prefilling.req.talker_out > 0:
                    talker_wait.append(prefilling)
                prefilling = None
        for s in stepped:
            s.decoded += 1
        still = []
        for s in decoding:
            if s.decoded >= s.req.backbone_out:
                engine.free("a", s.req.rid)
                if down_finished(s):
                    s.t_done = t
                    done.append(s)
            else:
                still.append(s)
        decoding = still
        still = []
        for s in talking:
            s.talker_done += 1
            if s.t_first_down is None:
                s.t_first_down = t
            if s.talker_done >= s.req.talker_out:
                engine.free("b", s.req.rid)
                if s.decoded >= s.req.backbone_out:
                    s.t_done = t
                    done.append(s)
            else:
                still.append(s)
        talking = still
        still = []
        for s in denoising:
            s.dit_done += 1
            if s.t_first_down is None:
                s.t_first_down = t
            if s.dit_done >= cfg.dit_steps:
                engine.free("c", s.req.rid)
                if s.decoded >= s.req.backbone_out:
                    s.t_done = t
                    done.append(s)
            else:
                still.append(s)
        denoising = still

    def pct(v, q):
        return float(np.percentile(v, q)) if v else None

    by_class = {}
    for cls in ("text", "speech", "image"):
        sel = [s for s in done if s.req.out_class == cls]
        ttft = [(s.t_first - s.req.arrival_s) * 1e3 for s in sel if s.t_first is not None]
        ttfo = [(s.t_first_down - s.req.arrival_s) * 1e3 for s in sel if s.t_first_down is not None]
        first = [(s.t_first if cls == "text" else s.t_first_down) for s in sel]
        met = [f is not None and (f - s.req.arrival_s) * 1e3 <= slo[cls] for f, s in zip(first, sel)]
        by_class[cls] = {"requests": len(sel), "ttft_ms_p50": pct(ttft, 50), "ttft_ms_p95": pct(ttft, 95),
                         "slo_ms": slo[cls], "slo_attainment": (sum(met) / len(met)) if met else None,
                         "first_downstream_ms_p50": pct(ttfo, 50), "first_downstream_ms_p95": pct(ttfo, 95)}
    if ctl is not None:
        ctl.close()
    if view is not None:
        view.close()
    return {"requests_done": len(done), "virtual_seconds": t, "busy_seconds": busy_s, "policy": cfg.policy,
            "pressure": {"mean": statistics.fmean(pressures) if pressures else None, "p95": pct(pressures, 95)},
            "cap_changes": cap_changes,
            "backbone_tokens": backbone_tokens, "talker_tokens": talker_tokens,
            "backbone_tokens_per_s": backbone_tokens / busy_s if busy_s else None,
            "tick_ms_by_budget": {str(b): {"n": len(v), "mean": statistics.fmean(v), "p50": pct(v, 50), "p95": pct(v, 95)}
                                  for b, v in sorted(ticks_by_budget.items(), reverse=True)},
            "talker_ms": {"n": len(talker_lat), "mean": statistics.fmean(talker_lat) if talker_lat else None,
                          "p95": pct(talker_lat, 95)},
            "image_stage": cfg.image_stage if use_dit else "talker", "dit_tokens": dit_tokens,
            "dit_ms": {"n": len(dit_lat), "mean": statistics.fmean(dit_lat) if dit_lat else None, "p95": pct(dit_lat, 95)},
            "by_class": by_class}


def pool_sizes(cfg: ReplayConfig, max_prompt: int = 4096, max_out: int = 512, max_talker_out: int = 1500):
    mpps_a = -(-(max_prompt + max_out + 1) // 16)
    mpps_b = -(-(cfg.talker_ctx0 + max_talker_out + 1) // 16)
    return (cfg.max_decode + 1) * mpps_a, cfg.max_talker * mpps_b, mpps_a, mpps_b


def main():
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--rate", type=float, default=8.0, help="Poisson arrival rate, requests per second")
    ap.add_argument("--requests", type=int, default=2000)
    ap.add_argument("--backbone", default="c3_7b")
    ap.add_argument("--talker", default="c4_talker")
    ap.add_argument("--policy", default="seeded", choices=["seeded", "controller", "horizon"])
    ap.add_argument("--b-sat", type=float, default=ReplayConfig.b_sat)
    ap.add_argument("--image-stage", default="talker", choices=["talker", "dit"],
                    help="downstream stage of the image class: talker-shaped steps, or the denoising stage (c6_dit)")
    args = ap.parse_args()
    cfg = ReplayConfig(policy=args.policy, b_sat=args.b_sat, image_stage=args.image_stage)
    pa, pb, ma, mb = pool_sizes(cfg)
    eng = GpuEngine(wl.DIMS[args.backbone], wl.DIMS[args.talker], pa, pb, ma, mb, cfg,
                    dims_c=wl.DIMS["c6_dit"] if args.image_stage == "dit" else None)
    try:
        res = replay(wl.make_trace(args.rate, args.requests), eng, cfg)
    finally:
        eng.close()
    res.update({"rate_per_s": args.rate, "backbone": args.backbone, "talker": args.talker})
    print(json.dumps(res))


if __name__ == "__main__":
    main()
