#!/usr/bin/env python
"""Benchmark of the shared-stage step: tokens/s and step latency under an SM budget, with the fraction of
the tensor-core roofline reached by the dominant kernel and the CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload c2_shared|c3_7b|c4_talker|c6_dit|c1_tiny] [--sm-budget B]

A "step" is one hs_stage_step over the whole batch (every layer: RMSNorm, QKV GEMM + RoPE + cache write,
paged attention, out-proj, gate/up + SwiGLU, down).  Inputs are seeded and synthetic.  With N > 1 (one
process per GPU under torch.distributed.run) every rank runs an independent replica of the same workload:
the step has no exchange between GPUs, so the data path uses no collective; ranks meet only at the timing
barriers.  `--impl reference` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_01785_b200 import workloads as wl  # noqa: E402

METRIC = "shared_stage_tokens_per_s"
UNIT = "tokens/s"
SEED = {"c1_tiny": 0, "c2_shared": 1, "c3_7b": 2, "c4_talker": 3, "c3_decode": 2, "c6_dit": 5}
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one gate/up GEMM launch, from the ncu
# capture summarised in profiles/gemm_pair_gateup_c2_shared.md (None where no capture of that launch exists).
GATEUP_DRAM_TRAFFIC_BYTES = {"c2_shared": 69989376 + 39707904}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def build_stage(name: str, device: int, init: str = "n002", layers: int = 0, flags: int = 0, batch=None):
    """Weights, KV pool with random-filled context, block tables and input of the named workload (or of the
    workload's dimensions with another batch)."""
    from paper_2608_01785_b200.stage import Stage
    dims = wl.DIMS[name]
    if layers:
        dims = wl.StageDims(layers, dims.d_model, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.d_ffn,
                            dims.rms_eps, dims.rope_base)
    seed = SEED[name]
    batch = batch or wl.make_batch(name, seed)
    dev = torch.device("cuda", device)
    weights = wl.make_weights(dims, seed, dev, init)
    num_pages = wl.pages_needed(batch) + 8
    mpps = max(-(-t // 16) for t in batch.total_len())
    stage = Stage(dims, weights, num_pages, batch.n_tokens, batch.n_seqs, mpps, max(batch.total_len()), device,
                  flags | wl.STAGE_FLAGS.get(name, 0))
    # context of the decode sequences: values do not change the timing; N(0,1) bf16 stands in for K/V
    # written by earlier steps
    g = torch.Generator(device=dev)
    g.manual_seed(seed + 1000)
    chunk = 1 << 24
    flat = stage.kv_pool
    for o in range(0, flat.numel(), chunk):
        n = min(chunk, flat.numel() - o)
        flat[o:o + n] = torch.randn(n, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    tables = [stage.kv_alloc(s, t) for s, t in enumerate(batch.total_len())]
    bt = stage.block_table_array(tables)
    x = wl.make_x(batch.n_tokens, dims.d_model, seed, dev)
    if name in wl.CONDITIONED:
        stage.set_modulation(wl.make_modulation(dims, batch.n_seqs, seed, dev))
    return stage, dims, batch, bt, x


def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's device-timed duration: replicas are independent, the job is as slow as its slowest."""
    if world <= 1:
        return ms
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(tokens_per_rank: int, world: int, ms_step_max: float) -> float:
    """Whole-job throughput of `world` replicas that each process tokens_per_rank tokens per step."""
    return world * tokens_per_rank / (ms_step_max * 1e-3)


def flops_per_step(dims: wl.StageDims, batch: wl.BatchSpec):
    T = batch.n_tokens
    gemm = 2.0 * T * dims.params_per_layer() * dims.n_layers
    attn = 0.0
    for n, c in zip(batch.q_len, batch.ctx_len):
        attn += 4.0 * dims.n_q_heads * dims.head_dim * (c * n + n * (n + 1) / 2.0)
    return gemm, attn * dims.n_layers


def cpu_oracle_sample(name: str, target_s: float):
    """Times the oracle on a bounded sample: one layer of the workload's batch, K/V of every token plus
    `rows` fully evaluated rows.  Returns (tokens/s extrapolated to the whole step, description, threads)."""
    from oracle.oracle import Oracle, OracleConfig
    from oracle.paging import PageAllocator, block_table_array
    dims = wl.DIMS[name]
    seed = SEED[name]
    batch = wl.make_batch(name, seed)
    one = wl.StageDims(1, dims.d_model, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.d_ffn)
    num_pages = wl.pages_needed(batch) + 8
    alloc = PageAllocator(num_pages, 16)
    tables = [alloc.alloc(s, t) for s, t in enumerate(batch.total_len())]
    bt = block_table_array(tables, max(len(t) for t in tables))
    cfg = OracleConfig(1, dims.d_model, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.d_ffn, 16, num_pages,
                       dims.rms_eps, dims.rope_base, bool(wl.STAGE_FLAGS.get(name, 0) & 2))
    w = wl.weights_to_numpy([wl.make_layer_weights(one, seed, 0)])
    if name in wl.CONDITIONED:
        w[0]["mod"] = wl.make_modulation(one, batch.n_seqs, seed)[0].numpy()
    pool = wl.bf16_bits_numpy(wl.make_kv_fill(one, num_pages, seed)).reshape(-1).copy()
    x = wl.to_f32_numpy(wl.make_x(batch.n_tokens, dims.d_model, seed))
    orc = Oracle("f32")
    T = batch.n_tokens
    # ~2 * params flops per fully evaluated row; the plain loops run at a few tens of GFLOP/s
    rows = int(max(16, min(T, target_s * 40e9 / (2.0 * dims.params_per_layer()))))
    mask = np.zeros(T, dtype=np.uint8)
    mask[np.linspace(0, T - 1, rows).astype(np.int64)] = 1
    rows = int(mask.sum())
    t0 = time.perf_counter()
    orc.step(cfg, w, pool, batch.q_len, batch.ctx_len, bt, x, mask)
    dt = time.perf_counter() - t0
    value = rows / (dt * dims.n_layers)
    desc = (f"one layer of {dims.n_layers}, batch of {name}: K/V of all {T} tokens + {rows} evenly spaced rows "
            f"evaluated in full, {dt:.2f} s; tokens/s = rows / (seconds x layers)")
    threads = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    return value, desc, threads, dt


def run_reference(args, rank: int):
    if rank != 0:
        return
    name = args.workload
    per_step = max(1.0, min(20.0, 150.0 / (args.steps + args.warmup)))
    for _ in range(args.warmup):
        cpu_oracle_sample(name, per_step)
    vals, times, desc, threads = [], [], "", 1
    for _ in range(args.steps):
        v, desc, threads, dt = cpu_oracle_sample(name, per_step)
        vals.append(v); times.append(dt)
    value = len(vals) / sum(1.0 / v for v in vals)          # harmonic mean = total tokens / total time
    dims, batch = wl.DIMS[name], wl.make_batch(name, SEED[name])
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * batch.n_tokens / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": name, "n_tokens": batch.n_tokens, "n_seqs": batch.n_seqs,
                       "n_layers": dims.n_layers},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_head(args):
    """Auxiliary measurement (not the headline metric): the sampling head behind a config-3 step -- final
    RMSNorm on the last row of each of the 65 sequences, the 152064 x 3584 vocabulary projection and the
    row-wise argmax -- and the embedding lookup in front of it.  HBM-bound: the vocabulary matrix is read once."""
    from paper_2608_01785_b200 import binding as B
    dev = torch.device("cuda", 0)
    d, V, n, T = wl.DIMS["c3_7b"].d_model, 152064, 65, 2112
    g = torch.Generator(device="cpu").manual_seed(11)
    y = torch.randn(T, d, generator=g).to(dev)
    gain = (1.0 + 0.02 * torch.randn(d, generator=g)).to(torch.bfloat16).to(dev)
    w = (0.02 * torch.randn(V, d, device=dev)).to(torch.bfloat16)
    rows = torch.arange(T - n, T, dtype=torch.int32, device=dev)
    cfg = B.make_head_config(d, V, 1e-6, 128)
    ws = torch.empty(B.hs_head_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
    head = B.hs_head_create(cfg, gain.data_ptr(), w.data_ptr(), ws.data_ptr())
    logits = torch.empty(n, V, device=dev)
    tokens = torch.empty(n, dtype=torch.int32, device=dev)
    x_emb = torch.empty(n, d, dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    budget = args.sm_budget or torch.cuda.get_device_properties(dev).multi_processor_count
    stream = torch.cuda.Stream(device=dev)

    def one():
        B.hs_head_step(head, y.data_ptr(), rows.data_ptr(), n, logits.data_ptr(), tokens.data_ptr(), budget,
                       stream.cuda_stream)
        B.hs_op_embed(tokens.data_ptr(), n, w.data_ptr(), V, d, x_emb.data_ptr(), budget, status.data_ptr(),
                      stream.cuda_stream)

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            one()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            one()
        e1.record(stream)
    torch.cuda.synchronize()
    assert B.hs_head_status(head) == 0 and status.item() == 0
    ms = e0.elapsed_time(e1) / args.steps
    B.hs_head_destroy(head)
    peaks = measured_peaks()
    bytes_moved = V * d * 2 + n * V * 4 * 2                     # the matrix once, the logits written and read
    print(json.dumps({"metric": "sampled_tokens_per_s", "value": n / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
                      "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
                      "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "c3_head", "d_model": d, "vocab": V, "rows": n, "sm_budget": budget,
                                 "l2": "the 1.09 GB vocabulary matrix exceeds L2"},
                      "roofline": {"bound": "hbm", "kernel": "head step (rmsnorm + vocabulary GEMM + argmax) + embed",
                                   "achieved": bytes_moved / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": bytes_moved / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_shared", choices=sorted(SEED) + ["c3_head"])
    ap.add_argument("--sm-budget", type=int, default=0, help="0 = all SMs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--bf16-activations", action="store_true",
                    help="stage flag HS_FLAG_BF16_ACTIVATIONS: h, o, act in bf16, no fp16 weight copies")
    ap.add_argument("--no-sweep", action="store_true", help="skip the SM-budget sweep and the co-run section")
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: cut the workload's stage to this many layers (not a benchmark configuration)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation of the step")
    if args.workload == "c3_head":
        if rank == 0:
            run_head(args)
        return

    import torch.distributed as dist
    from paper_2608_01785_b200 import binding as B
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    name = args.workload
    stage, dims, batch, bt, x = build_stage(name, local_rank, layers=args.layers, flags=1 if args.bf16_activations else 0)
    budget = args.sm_budget or stage.sm_count
    T, d = batch.n_tokens, dims.d_model
    dev = stage.device
    y = torch.empty(T, d, dtype=torch.float32, device=dev)
    b = stage.make_batch(batch.q_len, batch.ctx_len, bt, x, y)
    stream = torch.cuda.Stream(device=dev)

    def timed_steps(k: int, fn):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(k):
                fn()
            e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, dev)

    step_dev = lambda: stage.step(b, budget, stream)

    # ---- device-resident throughput -------------------------------------
    timed_steps(args.warmup, step_dev)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ms_total = timed_steps(args.steps, step_dev)
    clocks = sampler.stop() if rank == 0 else None
    assert stage.status() == 0, "device status word is set"
    ms_step = ms_total / args.steps
    value = aggregate_tokens_per_s(T, world, ms_step)

    # ---- per-kernel timing (same launches, events around each kernel) ----
    B.hs_stage_profile_enable(stage.handle, True)
    timed_steps(args.steps, step_dev)
    prof = B.hs_stage_profile_read(stage.handle)
    B.hs_stage_profile_enable(stage.handle, False)
    launches_per_step = sum(n for _, n in prof.values()) // args.steps

    # ---- end to end: host buffers in, host buffers out -------------------
    # Every step's x_in comes from pinned host memory and its y_out goes back to pinned host memory, all
    # inside the timed region.  The copies of step i+1 / i-1 run on their own streams beside the kernels of
    # step i (two device buffers each way), as a serving loop would do it.
    x_host = x.cpu().pin_memory()
    y_host = torch.empty(T, d, dtype=torch.float32).pin_memory()
    x_dev2 = [torch.empty_like(x) for _ in range(2)]
    y_dev2 = [torch.empty(T, d, dtype=torch.float32, device=dev) for _ in range(2)]
    b2 = [stage.make_batch(batch.q_len, batch.ctx_len, bt, x_dev2[i], y_dev2[i]) for i in range(2)]
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    def e2e_steps(k: int) -> float:
        barrier()
        in_done = [torch.cuda.Event() for _ in range(k)]
        cmp_done = [torch.cuda.Event() for _ in range(k)]
        out_done = [torch.cuda.Event() for _ in range(k)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s_in)
        for i in range(k):
            j = i & 1
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(cmp_done[i - 2])        # x_dev2[j] was read by step i-2
                x_dev2[j].copy_(x_host, non_blocking=True)
                in_done[i].record(s_in)
            stream.wait_event(in_done[i])
            if i >= 2:
                stream.wait_event(out_done[i - 2])          # y_dev2[j] has been copied out
            stage.step(b2[j], budget, stream)
            cmp_done[i].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(cmp_done[i])
                y_host.copy_(y_dev2[j], non_blocking=True)
                out_done[i].record(s_out)
        e1.record(s_out)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, dev)

    e2e_steps(3)
    ms_e2e = e2e_steps(args.steps) / args.steps
    e2e_value = aggregate_tokens_per_s(T, world, ms_e2e)

    # ---- step latency vs SM budget, and the co-run with a downstream stage (rank 0, single GPU) ----
    sweep, corun_rows, corun_dit_rows = None, None, None
    if rank == 0 and world == 1 and not args.no_sweep:
        sweep = []
        for bud in [x for x in wl.SM_BUDGETS.get(name, (148, 112, 74, 37)) if x <= stage.sm_count]:
            fn = lambda: stage.step(b, bud, stream)
            timed_steps(3, fn)
            ms_b = timed_steps(args.steps, fn) / args.steps
            sweep.append({"sm_budget": bud, "ms_per_step": ms_b, "tokens_per_s": T / (ms_b * 1e-3)})
        for row in sweep:
            row["speed_vs_full"] = sweep[0]["ms_per_step"] / row["ms_per_step"]
            row["budget_fraction"] = row["sm_budget"] / sweep[0]["sm_budget"]
        if name == "c2_shared":
            from paper_2608_01785_b200.corun import corun
            talker, tdims, tbatch, tbt, tx = build_stage("c4_talker", local_rank)
            ty = torch.empty(tbatch.n_tokens, tdims.d_model, dtype=torch.float32, device=dev)
            tb = talker.make_batch(tbatch.q_len, tbatch.ctx_len, tbt, tx, ty)
            corun_rows = [corun(stage, b, talker, tb, bud, args.steps) for bud in wl.SM_BUDGETS["c4_corun"]]
            assert talker.status() == 0
            talker.close()
            # the same co-run with the denoising-style stage (the image path's downstream partner)
            dit, ddims, dbatch, dbt, dx = build_stage("c6_dit", local_rank)
            dy = torch.empty(dbatch.n_tokens, ddims.d_model, dtype=torch.float32, device=dev)
            db = dit.make_batch(dbatch.q_len, dbatch.ctx_len, dbt, dx, dy)
            corun_dit_rows = [corun(stage, b, dit, db, bud, max(args.steps // 4, 5)) for bud in wl.SM_BUDGETS["c4_corun"]]
            assert dit.status() == 0
            dit.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (gate/up GEMM) -------------------
    peaks = measured_peaks()
    gu_ms, gu_n = prof["gemm_gateup"]
    gu_flops = 2.0 * T * dims.d_model * 2 * dims.d_ffn
    gu_avg_s = gu_ms * 1e-3 / max(gu_n, 1)
    achieved = gu_flops / gu_avg_s / 1e12
    peak = peaks["bf16_sustained"] * budget / stage.sm_count
    gemm_flops, attn_flops = flops_per_step(dims, batch)
    gateup_kernel = ("gemm_pair_kernel" if T > 128 and budget >= 2 else
                     "gemm_kernel" if T > 64 else "gemm_kernel or gemm_skinny_kernel (chosen by shape)")
    roofline = {"bound": "tensor", "kernel": gateup_kernel + " (gate/up + SwiGLU epilogue)", "achieved": achieved,
                "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_source": f"{peaks['source']} sustained bf16 (fp16 operands: nominal ratio 1.0) x sm_budget/{stage.sm_count}",
                "frac_of_burst_peak": achieved / (peaks["bf16_burst"] * budget / stage.sm_count),
                "traffic": GATEUP_DRAM_TRAFFIC_BYTES.get(name),
                "avg_launch_ms": gu_avg_s * 1e3, "launches": gu_n,
                "step_tflops": (gemm_flops + attn_flops) / (ms_step * 1e-3) / 1e12}
    kernels = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps} for k, v in prof.items()}
    # decode attention against HBM: K and V pages of every decode sequence once per layer
    dec_ms, dec_n = prof["attn_decode"]
    dec_bytes = sum((c + 1) * 2 * dims.kv_dim * 2 for q, c in zip(batch.q_len, batch.ctx_len) if q == 1)
    decode_roofline = None
    if dec_n:
        gbs = dec_bytes / (dec_ms * 1e-3 / dec_n) / 1e9
        decode_roofline = {"bound": "hbm", "kernel": "attn_decode_kernel", "achieved": gbs,
                           "peak": peaks["hbm_gbs"] * budget / stage.sm_count, "unit": "GB/s",
                           "frac": gbs / (peaks["hbm_gbs"] * budget / stage.sm_count),
                           "bytes_per_launch": dec_bytes, "avg_launch_ms": dec_ms / dec_n,
                           "note": "bytes below the 126 MB L2 are served from L2, not HBM" if dec_bytes < 126e6 else
                                   "working set exceeds L2"}

    cpu = None
    if not args.no_cpu_baseline:
        v, desc, threads, _ = cpu_oracle_sample(name, 12.0)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": name + (f" (cut to {args.layers} layers: profiling only)" if args.layers else ""),
                       "n_layers": dims.n_layers, "d_model": d, "n_tokens": T,
                       "n_seqs": batch.n_seqs, "prefill_tokens": int(sum(q for q in batch.q_len if q > 1)),
                       "decode_seqs": int(sum(1 for q in batch.q_len if q == 1)), "sm_budget": budget,
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                       "l2": "inputs larger than L2: weights + KV read per step exceed the 126 MB L2",
                       "formats": "all-bf16 operands (HS_FLAG_BF16_ACTIVATIONS); fp32 accumulation" if
                                  args.bf16_activations else
                                  "bf16 x_in, weights, KV cache, q and softmax weights; fp16 h, o, act against fp16 "
                                  "copies of the weights; fp32 accumulation, residual stream and output"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e, "h2d_bytes_per_step": T * d * 2,
                    "d2h_bytes_per_step": T * d * 4},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "roofline_decode_attention": decode_roofline, "kernels": kernels,
            "budget_sweep": sweep, "corun": corun_rows, "corun_dit": corun_dit_rows, "cpu_baseline": cpu}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
