#!/usr/bin/env python
"""Writes tests/golden/c3_end_to_end.npz: the CPU oracle's output of the whole 28-layer config-3 step on sampled
rows, for the GPU test that compares the library's step with it end to end.

Calls only the oracle and the seeded input generators (drawn on the CPU, so that the GPU test can draw the very
same buffers and upload them).  Inputs: the config-3 batch (one 2048-token prefill chunk + 64 decode sequences with
512..4096 cached tokens, seed 2), weights with the depth-scaled output projections (config 3 names no
distribution; std 0.02 and, for w_o / w_down, 0.02 / sqrt(2 L)), each layer's cache context filled with bf16
N(0,1) from a per-layer sub-stream.  Layers 0..26 are evaluated for every row (the next layer's K / V need them),
the last layer for the sampled rows only.

About a quarter of an hour on 8 cores, 8 GB of memory:  python tests/golden/make_c3_end_to_end.py
"""
import os
import sys
import time
import zlib

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle.oracle import Oracle, OracleConfig          # noqa: E402
from oracle.paging import PageAllocator, block_table_array          # noqa: E402
from paper_2608_01785_b200 import workloads as wl       # noqa: E402

NAME, SEED, INIT = "c3_7b", 2, "depth_scaled"
OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c3_end_to_end.npz")


def sampled_rows(batch) -> np.ndarray:
    """First / last rows of the prefill chunk, both sides of the 16-, 128- and 256-row tile edges, an even spread,
    and every fourth decode row (and the last one)."""
    n_pre = batch.q_len[0]
    edges = [0, 1, 15, 16, 17, 127, 128, 129, 255, 256, 257, 1023, 1024, 2031, 2032, n_pre - 2, n_pre - 1]
    spread = np.linspace(0, n_pre - 1, 40).astype(np.int64)
    dec = np.arange(n_pre, batch.n_tokens, 4)
    return np.unique(np.concatenate([np.array(edges), spread, dec, np.array([batch.n_tokens - 1])]))


def case_layout(dims, batch):
    """Pool size, block tables: the library's allocator hands out the same pages (pops 0, 1, 2, ...)."""
    num_pages = wl.pages_needed(batch) + 8
    alloc = PageAllocator(num_pages, 16)
    tables = [alloc.alloc(s, t) for s, t in enumerate(batch.total_len())]
    mpps = max(len(t) for t in tables)
    return num_pages, block_table_array(tables, mpps)


def crc(a: np.ndarray) -> int:
    return zlib.crc32(np.ascontiguousarray(a).view(np.uint8).reshape(-1).data) & 0xFFFFFFFF


def main():
    dims = wl.DIMS[NAME]
    batch = wl.make_batch(NAME, SEED)
    num_pages, bt = case_layout(dims, batch)
    rows = sampled_rows(batch)
    cfg1 = OracleConfig(1, dims.d_model, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.d_ffn, 16, num_pages,
                        dims.rms_eps, dims.rope_base)
    orc = Oracle("f32")
    x_t = wl.make_x(batch.n_tokens, dims.d_model, SEED)
    x = wl.to_f32_numpy(x_t)
    checks = {"x": crc(wl.bf16_bits_numpy(x_t))}
    t0 = time.time()
    for layer in range(dims.n_layers):
        w_t = wl.make_layer_weights(dims, SEED, layer, "cpu", INIT)
        pool_t = wl.make_kv_fill_layer(dims, num_pages, SEED, layer)
        if layer in (0, dims.n_layers - 1):
            checks[f"w_down_{layer}"] = crc(wl.bf16_bits_numpy(w_t["w_down"]))
            checks[f"kv_{layer}"] = crc(wl.bf16_bits_numpy(pool_t))
        w = {k: wl.to_f32_numpy(v) for k, v in w_t.items()}
        pool = wl.bf16_bits_numpy(pool_t).reshape(-1).copy()
        del w_t, pool_t
        mask = None
        if layer == dims.n_layers - 1:
            mask = np.zeros(batch.n_tokens, dtype=np.uint8)
            mask[rows] = 1
        x, _ = orc.layer(cfg1, w, 0, pool, batch.q_len, batch.ctx_len, bt, x, row_mask=mask)
        rms = float(np.sqrt(np.mean(x[rows].astype(np.float64) ** 2)))
        print(f"layer {layer:2d} done, {time.time() - t0:6.0f} s, RMS of the sampled rows {rms:.4f}", flush=True)
    np.savez_compressed(OUT, rows=rows.astype(np.int32), y=x[rows].astype(np.float32),
                        input_crc32=np.array([[k, str(v)] for k, v in sorted(checks.items())]),
                        recipe=np.array([NAME, str(SEED), INIT, str(num_pages)]))
    print("wrote", OUT, os.path.getsize(OUT), "bytes")


if __name__ == "__main__":
    main()
