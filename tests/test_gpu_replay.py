"""Trace replay on real stages (small dimensions): the backbone and the talker are stepped through the C
ABI on two streams with complementary SM budgets, tick after tick, with sequences joining and leaving."""
import pytest

from paper_2608_01785_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("policy", ["seeded", "controller"])
def test_replay_small_trace_on_gpu(policy):
    from paper_2608_01785_b200.replay import GpuEngine, ReplayConfig, pool_sizes, replay
    cfg = ReplayConfig(max_decode=12, max_prefill_chunk=512, max_talker=4, ladder=(120, 96, 74, 48), policy=policy,
                       b_sat=0.02)          # small stages move few bytes: a low saturation point makes the cap move
    trace = [wl.Request(r.rid, r.arrival_s, r.out_class, min(r.prompt_len, 900), min(r.backbone_out, 40),
                        min(r.talker_out, 60)) for r in wl.make_trace(16.0, 30, seed=4)]
    pa, pb, ma, mb = pool_sizes(cfg, max_prompt=900, max_out=40, max_talker_out=60)
    backbone = wl.StageDims(2, 512, 8, 2, 64, 1408)
    talker = wl.StageDims(2, 256, 4, 2, 64, 688)
    eng = GpuEngine(backbone, talker, pa, pb, ma, mb, cfg)
    try:
        res = replay(trace, eng, cfg)
        assert res["requests_done"] == 30
        assert res["backbone_tokens"] == sum(r.prompt_len + r.backbone_out for r in trace)
        assert res["talker_tokens"] == sum(r.talker_out for r in trace)
        assert eng.free_pages("a") == pa and eng.free_pages("b") == pb
        assert res["backbone_tokens_per_s"] > 0
        assert set(res["tick_ms_by_budget"]) <= {"148", "120", "96", "74", "48"}
    finally:
        eng.close()


def test_replay_with_the_denoising_stage_on_gpu():
    """The image class on a real third stage (no causal mask, conditioned): every image gets its denoising steps,
    the talker only sees the speech class, and the three page pools return to empty."""
    from paper_2608_01785_b200.replay import GpuEngine, ReplayConfig, pool_sizes, replay
    cfg = ReplayConfig(max_decode=12, max_prefill_chunk=512, max_talker=4, policy="controller", b_sat=0.02,
                       image_stage="dit", dit_steps=5, dit_tokens=96, max_dit=3)
    trace = [wl.Request(r.rid, r.arrival_s, r.out_class, min(r.prompt_len, 900), min(r.backbone_out, 40),
                        min(r.talker_out, 60)) for r in wl.make_trace(16.0, 30, seed=4)]
    pa, pb, ma, mb = pool_sizes(cfg, max_prompt=900, max_out=40, max_talker_out=60)
    backbone = wl.StageDims(2, 512, 8, 2, 64, 1408)
    talker = wl.StageDims(2, 256, 4, 2, 64, 688)
    dit = wl.StageDims(2, 256, 4, 4, 64, 688)
    eng = GpuEngine(backbone, talker, pa, pb, ma, mb, cfg, dims_c=dit)
    try:
        res = replay(trace, eng, cfg)
        n_img = sum(r.out_class == "image" for r in trace)
        assert n_img > 0 and res["requests_done"] == 30 and res["image_stage"] == "dit"
        assert res["talker_tokens"] == sum(r.talker_out for r in trace if r.out_class == "speech")
        assert res["dit_tokens"] == n_img * cfg.dit_steps * cfg.dit_tokens
        assert eng.free_pages("a") == pa and eng.free_pages("b") == pb
        assert eng.free_pages("c") == cfg.max_dit * -(-cfg.dit_tokens // 16)
        assert res["dit_ms"]["mean"] > 0
    finally:
        eng.close()
