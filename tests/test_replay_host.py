"""Scheduling logic of the trace replay, on the latency-model engine (no GPU): every request finishes,
token counts are conserved, the page allocators of both stages return to empty, budgets come from the
ladder only while the talker has work."""
import numpy as np

from paper_2608_01785_b200 import workloads as wl
from paper_2608_01785_b200.replay import ModelEngine, ReplayConfig, pool_sizes, replay


def test_trace_statistics():
    tr = wl.make_trace(8.0, 2000, seed=4)
    assert len(tr) == 2000
    gaps = np.diff([0.0] + [r.arrival_s for r in tr])
    assert abs(gaps.mean() - 1 / 8.0) < 0.01                       # Poisson arrivals at the stated rate
    frac = {c: sum(r.out_class == c for r in tr) / 2000 for c in ("text", "speech", "image")}
    assert abs(frac["text"] - 0.3) < 0.04 and abs(frac["speech"] - 0.5) < 0.04 and abs(frac["image"] - 0.2) < 0.04
    p = np.array([r.prompt_len for r in tr])
    assert p.min() >= 64 and p.max() <= 4096 and 520 < np.median(p) < 690
    assert all(64 <= r.backbone_out <= 512 for r in tr)
    assert all((r.talker_out == 0) == (r.out_class == "text") for r in tr)
    assert all(200 <= r.talker_out <= 1500 for r in tr if r.out_class != "text")
    assert wl.make_trace(8.0, 50, seed=4)[:50] == tr[:50]           # seeded


def test_replay_conserves_tokens_and_pages():
    cfg = ReplayConfig(max_decode=8, max_prefill_chunk=256, max_talker=4)
    trace = wl.make_trace(16.0, 60, seed=4)
    pa, pb, ma, mb = pool_sizes(cfg)
    eng = ModelEngine(wl.DIMS["c1_tiny"], wl.DIMS["c1_tiny"], pa, pb, ma, mb)
    try:
        res = replay(trace, eng, cfg)
        assert res["requests_done"] == 60
        assert res["backbone_tokens"] == sum(r.prompt_len + r.backbone_out for r in trace)
        assert res["talker_tokens"] == sum(r.talker_out for r in trace)
        assert eng.free_pages("a") == pa and eng.free_pages("b") == pb      # everything was returned
        budgets = {int(b) for b in res["tick_ms_by_budget"]}
        assert budgets <= {148, *cfg.ladder} and 148 in budgets and budgets & set(cfg.ladder)
        for cls in ("text", "speech", "image"):
            c = res["by_class"][cls]
            assert c["requests"] == sum(r.out_class == cls for r in trace)
            assert c["ttft_ms_p50"] is not None and c["ttft_ms_p50"] > 0
        assert res["by_class"]["text"]["first_downstream_ms_p50"] is None
        assert res["by_class"]["speech"]["first_downstream_ms_p50"] >= res["by_class"]["speech"]["ttft_ms_p50"]
        assert res["virtual_seconds"] >= res["busy_seconds"] > 0
    finally:
        eng.close()


def test_replay_with_the_denoising_stage_for_images():
    """image_stage = "dit": images leave the talker's queue and run a fixed number of denoising steps on a third
    stage; talker tokens are then those of the speech class only, every image gets exactly dit_steps steps of
    dit_tokens tokens, and all three page pools return to empty."""
    cfg = ReplayConfig(max_decode=8, max_prefill_chunk=256, max_talker=4, image_stage="dit", dit_steps=7, dit_tokens=48,
                       max_dit=2)
    trace = wl.make_trace(16.0, 60, seed=4)
    pa, pb, ma, mb = pool_sizes(cfg)
    mc = -(-cfg.dit_tokens // 16)
    pc = cfg.max_dit * mc
    eng = ModelEngine(wl.DIMS["c1_tiny"], wl.DIMS["c1_tiny"], pa, pb, ma, mb, wl.DIMS["c1_tiny"], pc, mc)
    try:
        res = replay(trace, eng, cfg)
        n_img = sum(r.out_class == "image" for r in trace)
        assert n_img > 0 and res["requests_done"] == 60 and res["image_stage"] == "dit"
        assert res["talker_tokens"] == sum(r.talker_out for r in trace if r.out_class == "speech")
        assert res["dit_tokens"] == n_img * cfg.dit_steps * cfg.dit_tokens
        assert res["dit_ms"]["n"] >= n_img * cfg.dit_steps / cfg.max_dit
        assert eng.free_pages("a") == pa and eng.free_pages("b") == pb and eng.free_pages("c") == pc
        img = res["by_class"]["image"]
        assert img["first_downstream_ms_p50"] >= img["ttft_ms_p50"] > 0
    finally:
        eng.close()
    # without a third stage in the engine the option falls back to talker-shaped steps
    eng = ModelEngine(wl.DIMS["c1_tiny"], wl.DIMS["c1_tiny"], pa, pb, ma, mb)
    try:
        res = replay(trace, eng, cfg)
        assert res["image_stage"] == "talker" and res["talker_tokens"] == sum(r.talker_out for r in trace)
    finally:
        eng.close()


def test_replay_under_the_spatial_controller():
    """The same replay with the library's controller choosing the budget: while the talker has work the
    backbone never gets more than the top of the ladder, it gets all SMs when the talker is idle, the cap
    follows the pressure (higher b_sat -> lower caps), and tokens and pages are conserved as before."""
    trace = wl.make_trace(16.0, 60, seed=4)
    seen = {}
    for b_sat in (0.05, 1e6):
        cfg = ReplayConfig(max_decode=8, max_prefill_chunk=256, max_talker=4, policy="controller", b_sat=b_sat,
                           hbm_gbs=0.01)                 # a tiny "peak" so that the model engine's ticks register
        pa, pb, ma, mb = pool_sizes(cfg)
        eng = ModelEngine(wl.DIMS["c1_tiny"], wl.DIMS["c1_tiny"], pa, pb, ma, mb)
        try:
            res = replay(trace, eng, cfg)
            assert res["requests_done"] == 60 and res["policy"] == "controller"
            assert res["backbone_tokens"] == sum(r.prompt_len + r.backbone_out for r in trace)
            assert eng.free_pages("a") == pa and eng.free_pages("b") == pb
            budgets = {int(b): v["n"] for b, v in res["tick_ms_by_budget"].items()}
            assert set(budgets) <= {148, *cfg.ladder} and 148 in budgets
            assert res["pressure"]["mean"] > 0
            seen[b_sat] = budgets
        finally:
            eng.close()
    co = lambda d: {b: n for b, n in d.items() if b != 148}
    assert max(co(seen[0.05])) == 120            # saturated pressure: the top of the ladder, never beyond it
    assert set(co(seen[1e6])) == {48}            # negligible pressure: the bottom of the ladder


def test_replay_with_the_temporal_view_protects_short_path_requests():
    """"horizon" = temporal view (path rotation, slack guard, long-path cap) + spatial controller.  On the latency
    model near saturation the short-path class reaches its first token sooner and meets its deadline more often
    than under first-come-first-served admission; nothing is lost or leaked."""
    trace = wl.make_trace(1.0, 200, seed=4)
    out = {}
    for policy in ("controller", "horizon"):
        cfg = ReplayConfig(max_decode=8, max_prefill_chunk=256, max_talker=4, policy=policy, hbm_gbs=0.01, long_cap=3,
                           slo_ms=(("text", 400.0), ("speech", 20000.0), ("image", 20000.0)))
        pa, pb, ma, mb = pool_sizes(cfg)
        eng = ModelEngine(wl.DIMS["c1_tiny"], wl.DIMS["c1_tiny"], pa, pb, ma, mb)
        try:
            res = replay(trace, eng, cfg)
            assert res["requests_done"] == 200
            assert res["backbone_tokens"] == sum(r.prompt_len + r.backbone_out for r in trace)
            assert res["talker_tokens"] == sum(r.talker_out for r in trace)
            assert eng.free_pages("a") == pa and eng.free_pages("b") == pb
            out[policy] = res["by_class"]
        finally:
            eng.close()
    assert out["horizon"]["text"]["ttft_ms_p95"] < out["controller"]["text"]["ttft_ms_p95"]
    assert out["horizon"]["text"]["slo_attainment"] >= out["controller"]["text"]["slo_attainment"]
    assert out["horizon"]["text"]["slo_attainment"] > 0.95
