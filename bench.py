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
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one gate/up GEMM launch per workload, each from one
# ncu capture of that launch (the config-3 launch was captured on a 2-layer cut of the stage: a layer's launch
# reads its own weights and the step's activations whatever the depth).  None where no capture exists.
GATEUP_DRAM_TRAFFIC_BYTES = {"c2_shared": 70058496 + 39722496, "c3_7b": 287605760 + 71187200}
# Below this length of the timed region a kernel runs at burst clocks and is held against the burst peak; a longer
# region settles under the power cap and is held against the sustained peak.
BURST_REGION_MS = 1000.0


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
                                          "--format=csv,noheader,nounits", "-lms", "20"],
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
    # a short calibration pass, then a sample sized for about target_s seconds of wall time: more rows of the layer,
    # and when the whole layer is not enough, the layer repeated
    def run(rows):
        mask = np.zeros(T, dtype=np.uint8)
        mask[np.linspace(0, T - 1, rows).astype(np.int64)] = 1
        t0 = time.perf_counter()
        orc.step(cfg, w, pool.copy(), batch.q_len, batch.ctx_len, bt, x, mask)
        return int(mask.sum()), time.perf_counter() - t0
    rows0, dt0 = run(max(16, min(T, T // 16)))
    rows = int(max(16, min(T, rows0 * target_s / max(dt0, 1e-3))))
    reps = 1
    if rows == T:
        reps = int(max(1, min(8, round(target_s / max(dt0 * T / rows0, 1e-3)))))
    done, dt = 0, 0.0
    for _ in range(reps):
        r, d = run(rows)
        done += r
        dt += d
    value = done / (dt * dims.n_layers)
    desc = (f"one layer of {dims.n_layers}, batch of {name}: K/V of all {T} tokens + {done // reps} evenly spaced rows "
            f"evaluated in full" + (f", {reps} times" if reps > 1 else "") +
            f", {dt:.2f} s; tokens/s = rows / (seconds x layers)")
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


def gemm_classes(dims: wl.StageDims, T: int):
    """flops = 2 M K N of the four projection launches of one layer."""
    d, F = dims.d_model, dims.d_ffn
    return {"gemm_qkv": 2.0 * T * d * (dims.q_dim + 2 * dims.kv_dim), "gemm_out": 2.0 * T * dims.q_dim * d,
            "gemm_gateup": 2.0 * T * d * 2 * F, "gemm_down": 2.0 * T * F * d}


def rooflines(name, dims, batch, prof, steps, ms_step, clocks, budget, sm_count, peaks):
    """Roofline entries from the per-class event timing: one per GEMM class, prefill attention (tensor), decode
    attention and RMSNorm (HBM).  The tensor peak is the burst figure when the timed region is short, the
    sustained one otherwise; both fractions are printed, and time x median SM clock lets a reader normalise."""
    T = batch.n_tokens
    region_ms = ms_step * steps
    use_burst = region_ms < BURST_REGION_MS
    peak_t = (peaks["bf16_burst"] if use_burst else peaks["bf16_sustained"]) * budget / sm_count
    mhz = (clocks or {}).get("sm_mhz")
    out = {}
    folded = prof["rmsnorm"][1] < prof["gemm_out"][1]      # fewer norm launches than layers: the residual GEMMs carry them
    for cls, flops in gemm_classes(dims, T).items():
        ms, n = prof[cls]
        if not n:
            continue
        avg_s = ms * 1e-3 / n
        ach = flops / avg_s / 1e12
        out[cls] = {"bound": "tensor", "achieved": ach, "peak": peak_t, "unit": "TFLOP/s", "frac": ach / peak_t,
                    "frac_of_burst_peak": ach / (peaks["bf16_burst"] * budget / sm_count),
                    "frac_of_sustained_peak": ach / (peaks["bf16_sustained"] * budget / sm_count),
                    "flops_per_launch": flops, "avg_launch_ms": avg_s * 1e3, "launches": n,
                    "ms_x_sm_mhz": avg_s * 1e3 * mhz if mhz else None}
        if folded and cls in ("gemm_out", "gemm_down"):
            out[cls]["note"] = ("this launch also does the RMSNorm that follows it (reads the residual stream, adds, writes it "
                                "back, emits the next GEMM's 16-bit operand and the rows' sums of squares); only the "
                                "projection's flops are counted")
    _, attn_flops = flops_per_step(dims, batch)
    ms, n = prof["attn_prefill"]
    if n:
        fl = attn_flops / dims.n_layers - sum(4.0 * dims.n_q_heads * dims.head_dim * (c + 1)
                                              for q, c in zip(batch.q_len, batch.ctx_len) if q == 1)
        ach = fl / (ms * 1e-3 / n) / 1e12
        out["attn_prefill"] = {"bound": "tensor", "achieved": ach, "peak": peak_t, "unit": "TFLOP/s", "frac": ach / peak_t,
                               "flops_per_launch": fl, "avg_launch_ms": ms / n, "launches": n,
                               "note": "causal flops 4 Hq Dh sum(c n + n (n + 1) / 2); bound by the exponentials "
                                       "as much as by the tensor pipe"}
    ms, n = prof["attn_decode"]
    if n:
        dec_bytes = sum((c + 1) * 2 * dims.kv_dim * 2 for q, c in zip(batch.q_len, batch.ctx_len) if q == 1)
        gbs = dec_bytes / (ms * 1e-3 / n) / 1e9
        out["attn_decode"] = {"bound": "hbm", "kernel": "attn_decode_kernel", "achieved": gbs, "peak": peaks["hbm_gbs"],
                              "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "bytes_per_launch": dec_bytes,
                              "avg_launch_ms": ms / n, "launches": n,
                              "note": ("K and V pages of every decode sequence once per layer; " +
                                       ("bytes below the 126 MB L2 are served from L2, not HBM" if dec_bytes < 126e6
                                        else "working set exceeds L2") + "; the HBM peak is not scaled by the budget")}
    ms, n = prof["rmsnorm"]
    if n:
        nbytes = T * dims.d_model * (4 + 2)
        gbs = nbytes / (ms * 1e-3 / n) / 1e9
        out["rmsnorm"] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                          "frac": gbs / peaks["hbm_gbs"], "bytes_per_launch": nbytes, "avg_launch_ms": ms / n, "launches": n}
    meta = {"timed_region_ms": region_ms, "tensor_peak_used": "burst" if use_burst else "sustained",
            "rule": f"burst peak when the timed region is under {BURST_REGION_MS:.0f} ms, sustained otherwise",
            "peaks": {"bf16_burst_tflops": peaks["bf16_burst"], "bf16_sustained_tflops": peaks["bf16_sustained"],
                      "hbm_gbs": peaks["hbm_gbs"], "source": peaks["source"]},
            "operands": "fp16 x fp16 (nominal rate equals bf16 x bf16: ratio 1.0)", "median_sm_mhz": mhz}
    return out, meta


class Measured:
    """Device-resident timing, per-class timing and the end-to-end leg of one workload on one stage."""

    def __init__(self, name, args, local_rank, rank, world, barrier, flags=0):
        self.name, self.args, self.rank, self.world, self.barrier = name, args, rank, world, barrier
        self.stage, self.dims, self.batch, self.bt, self.x = build_stage(name, local_rank, layers=args.layers, flags=flags)
        self.dev = self.stage.device
        self.T, self.d = self.batch.n_tokens, self.dims.d_model
        self.y = torch.empty(self.T, self.d, dtype=torch.float32, device=self.dev)
        self.b = self.stage.make_batch(self.batch.q_len, self.batch.ctx_len, self.bt, self.x, self.y)
        self.stream = torch.cuda.Stream(device=self.dev)
        self.budget = args.sm_budget or self.stage.sm_count

    def timed_steps(self, k, fn):
        self.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(self.stream):
            e0.record(self.stream)
            for _ in range(k):
                fn()
            e1.record(self.stream)
        self.barrier()
        return max_over_ranks(e0.elapsed_time(e1), self.world, self.dev)

    def step_fn(self, budget=None):
        bud = budget or self.budget
        return lambda: self.stage.step(self.b, bud, self.stream)

    def device_resident(self, steps, warmup, sample_clocks):
        self.timed_steps(warmup, self.step_fn())
        sampler = ClockSampler(self.dev.index or 0)
        if sample_clocks:
            # nvidia-smi needs a few hundred milliseconds to deliver its first sample; a short workload keeps
            # stepping (untimed) until it has, so that the samples are taken under this workload's load
            sampler.start()
            t_end = time.perf_counter() + 1.5
            while not sampler.lines and time.perf_counter() < t_end:
                self.timed_steps(max(warmup, 5), self.step_fn())
            sampler.lines.clear()
        ms_total = self.timed_steps(steps, self.step_fn())
        clocks = sampler.stop() if sample_clocks else None
        assert self.stage.status() == 0, "device status word is set"
        assert self.stage.saturation_count() == 0, "fp16 activations were clamped"
        return ms_total / steps, clocks

    def per_class(self, steps):
        from paper_2608_01785_b200 import binding as B
        B.hs_stage_profile_enable(self.stage.handle, True)
        self.timed_steps(steps, self.step_fn())
        prof = B.hs_stage_profile_read(self.stage.handle)
        B.hs_stage_profile_enable(self.stage.handle, False)
        return prof

    def e2e(self, steps):
        """Every step's x_in comes from pinned host memory and its y_out goes back to pinned host memory, all inside
        the timed region.  The copies of step i+1 / i-1 run on their own streams beside the kernels of step i (two
        device buffers each way), as a serving loop would do it."""
        stage, batch, bt, x, dev, T, d = self.stage, self.batch, self.bt, self.x, self.dev, self.T, self.d
        x_host = x.cpu().pin_memory()
        y_host = torch.empty(T, d, dtype=torch.float32).pin_memory()
        x_dev2 = [torch.empty_like(x) for _ in range(2)]
        y_dev2 = [torch.empty(T, d, dtype=torch.float32, device=dev) for _ in range(2)]
        b2 = [stage.make_batch(batch.q_len, batch.ctx_len, bt, x_dev2[i], y_dev2[i]) for i in range(2)]
        s_in, s_out, stream = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev), self.stream

        def run(k):
            self.barrier()
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
                stage.step(b2[j], self.budget, stream)
                cmp_done[i].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(cmp_done[i])
                    y_host.copy_(y_dev2[j], non_blocking=True)
                    out_done[i].record(s_out)
            e1.record(s_out)
            self.barrier()
            return max_over_ranks(e0.elapsed_time(e1), self.world, dev)

        run(3)
        return run(steps) / steps

    def sweep(self, steps):
        rows = []
        for bud in [x for x in wl.SM_BUDGETS.get(self.name, (148, 112, 74, 37)) if x <= self.stage.sm_count]:
            fn = self.step_fn(bud)
            self.timed_steps(3, fn)
            ms_b = self.timed_steps(steps, fn) / steps
            rows.append({"sm_budget": bud, "ms_per_step": ms_b, "tokens_per_s": self.T / (ms_b * 1e-3)})
        for row in rows:
            row["speed_vs_full"] = rows[0]["ms_per_step"] / row["ms_per_step"]
            row["budget_fraction"] = row["sm_budget"] / rows[0]["sm_budget"]
        return rows

    def close(self):
        self.stage.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3_7b", choices=sorted(SEED) + ["c3_head"])
    ap.add_argument("--sm-budget", type=int, default=0, help="0 = all SMs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--bf16-activations", action="store_true",
                    help="stage flag HS_FLAG_BF16_ACTIVATIONS: h, o, act in bf16, no fp16 weight copies")
    ap.add_argument("--no-sweep", action="store_true",
                    help="skip the SM-budget sweep, the all-bf16 leg and the config-2 / co-run section")
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
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    name = args.workload
    peaks = measured_peaks()
    m = Measured(name, args, local_rank, rank, world, barrier, flags=1 if args.bf16_activations else 0)
    dims, batch, T, d, budget, stage = m.dims, m.batch, m.T, m.d, m.budget, m.stage

    # ---- device-resident throughput, per-kernel timing, end to end -----------
    ms_step, clocks = m.device_resident(args.steps, args.warmup, rank == 0)
    value = aggregate_tokens_per_s(T, world, ms_step)
    prof = m.per_class(args.steps)
    launches_per_step = sum(n for _, n in prof.values()) // args.steps
    ms_e2e = m.e2e(args.steps)
    e2e_value = aggregate_tokens_per_s(T, world, ms_e2e)

    # ---- rank 0, single GPU: budget sweep, the all-bf16 form, config 2 and the co-runs ----
    sweep, bf16_leg, c2_obj, corun_rows, corun_dit_rows = None, None, None, None, None
    small = max(args.steps // 2, 5)
    if rank == 0 and world == 1 and not args.no_sweep:
        sweep = m.sweep(args.steps)
        if not args.bf16_activations and name in ("c3_7b", "c2_shared"):
            # the same step with every operand in bf16 (HS_FLAG_BF16_ACTIVATIONS: no fp16 copies of the weights)
            mb = Measured(name, args, local_rank, rank, world, barrier, flags=1)
            ms_b, _ = mb.device_resident(small, 3, False)
            bf16_leg = {"ms_per_step": ms_b, "tokens_per_s": T / (ms_b * 1e-3), "steps": small,
                        "formats": "all-bf16 operands (HS_FLAG_BF16_ACTIVATIONS); fp32 accumulation"}
            mb.close()
            del mb
        if name == "c3_7b":
            # config 2 (shared backbone, 4 layers) with its own sweep, per-class rooflines and the co-runs of config 4
            from paper_2608_01785_b200.corun import corun
            steps2 = max(args.steps, 20)
            m2 = Measured("c2_shared", args, local_rank, rank, world, barrier)
            ms2, clocks2 = m2.device_resident(steps2, 3, True)
            prof2 = m2.per_class(steps2)
            roof2, roof2_meta = rooflines("c2_shared", m2.dims, m2.batch, prof2, steps2, ms2, clocks2, m2.budget,
                                          m2.stage.sm_count, peaks)
            c2_obj = {"workload": "c2_shared", "n_tokens": m2.T, "n_layers": m2.dims.n_layers, "steps": steps2,
                      "ms_per_step": ms2, "tokens_per_s": m2.T / (ms2 * 1e-3), "e2e_ms_per_step": m2.e2e(steps2),
                      "clocks": clocks2, "rooflines": roof2, "roofline_basis": roof2_meta,
                      "kernels": {k: {"ms_per_step": v[0] / steps2, "launches_per_step": v[1] / steps2} for k, v in prof2.items()},
                      "budget_sweep": m2.sweep(steps2)}
            talker, tdims, tbatch, tbt, tx = build_stage("c4_talker", local_rank)
            ty = torch.empty(tbatch.n_tokens, tdims.d_model, dtype=torch.float32, device=m2.dev)
            tb = talker.make_batch(tbatch.q_len, tbatch.ctx_len, tbt, tx, ty)
            corun_rows = [corun(m2.stage, m2.b, talker, tb, bud, steps2) for bud in wl.SM_BUDGETS["c4_corun"]]
            assert talker.status() == 0
            talker.close()
            dit, ddims, dbatch, dbt, dx = build_stage("c6_dit", local_rank)
            dy = torch.empty(dbatch.n_tokens, ddims.d_model, dtype=torch.float32, device=m2.dev)
            db = dit.make_batch(dbatch.q_len, dbatch.ctx_len, dbt, dx, dy)
            corun_dit_rows = [corun(m2.stage, m2.b, dit, db, bud, max(steps2 // 4, 5)) for bud in wl.SM_BUDGETS["c4_corun"]]
            assert dit.status() == 0
            dit.close()
            m2.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- rooflines ---------------------------------------------------------
    roofs, roof_meta = rooflines(name, dims, batch, prof, args.steps, ms_step, clocks, budget, stage.sm_count, peaks)
    gemm_flops, attn_flops = flops_per_step(dims, batch)
    gateup_kernel = ("gemm_pair_kernel" if T > 128 and budget >= 2 else
                     "gemm_kernel" if T > 64 else "gemm_kernel or gemm_skinny_kernel (chosen by shape)")
    roofline = dict(roofs.get("gemm_gateup", {}))
    roofline.update({"kernel": gateup_kernel + " (gate/up + SwiGLU epilogue), the dominant kernel of the step",
                     "peak_source": f"{peaks['source']} {roof_meta['tensor_peak_used']} bf16 (timed region "
                                    f"{roof_meta['timed_region_ms']:.0f} ms; fp16 operands: nominal ratio 1.0) "
                                    f"x sm_budget/{stage.sm_count}",
                     "traffic": GATEUP_DRAM_TRAFFIC_BYTES.get(name) if not args.layers else None,
                     "algorithmic_bytes": T * d * 2 + 2 * dims.d_ffn * d * 2 + T * dims.d_ffn * 2,
                     "step_tflops": (gemm_flops + attn_flops) / (ms_step * 1e-3) / 1e12})
    kernels = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps} for k, v in prof.items()}

    cpu = None
    if not args.no_cpu_baseline:
        v, desc, threads, _ = cpu_oracle_sample(name, 12.0)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if args.bf16_activations else "f16", "data": "synthetic",
            "dtype_detail": "all-bf16 operands (HS_FLAG_BF16_ACTIVATIONS); fp32 accumulation" if args.bf16_activations else
                            "projections: fp16 x fp16 -> fp32 (h, o, act in fp16 against fp16 copies of the bf16 weights); "
                            "attention: bf16 x bf16 -> fp32 (q, K, V, softmax weights in bf16); fp32 residual stream and "
                            "output; bf16 x_in, weights and KV cache at the interface",
            "config": {"workload": name + (f" (cut to {args.layers} layers: profiling only)" if args.layers else ""),
                       "n_layers": dims.n_layers, "d_model": d, "n_tokens": T,
                       "n_seqs": batch.n_seqs, "prefill_tokens": int(sum(q for q in batch.q_len if q > 1)),
                       "decode_seqs": int(sum(1 for q in batch.q_len if q == 1)), "sm_budget": budget,
                       "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                       "l2": "inputs larger than L2: weights + KV read per step exceed the 126 MB L2"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e, "h2d_bytes_per_step": T * d * 2,
                    "d2h_bytes_per_step": T * d * 4},
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "rooflines": roofs, "roofline_basis": roof_meta,
            "roofline_decode_attention": roofs.get("attn_decode"), "kernels": kernels,
            "budget_sweep": sweep, "bf16_path": bf16_leg,
            "bf16_path_ms_per_step": bf16_leg["ms_per_step"] if bf16_leg else None,
            "c2_shared": c2_obj, "corun": corun_rows, "corun_dit": corun_dit_rows, "cpu_baseline": cpu}
    print(json.dumps(line))
    m.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
