"""Shared set-up for the tests: builds oracle-side cases from the seeded generators."""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np

from oracle.oracle import OracleConfig
from oracle.paging import PageAllocator, block_table_array
from paper_2608_01785_b200 import workloads as wl


@dataclass
class Case:
    dims: wl.StageDims
    cfg: OracleConfig
    weights: List[Dict[str, np.ndarray]]      # float32 views of the bf16 weights
    weights_t: list                           # the bf16 torch tensors themselves
    batch: wl.BatchSpec
    block_tables: np.ndarray                  # int32 [n_seqs, max_pages_per_seq]
    kv_pool: np.ndarray                       # uint16 bf16 bits, interface layout, flat
    x_t: object                               # bf16 torch tensor [T, d]
    x: np.ndarray                             # its float32 view

    @property
    def mpps(self) -> int:
        return self.block_tables.shape[1]


def oracle_cfg(dims: wl.StageDims, num_pages: int) -> OracleConfig:
    return OracleConfig(dims.n_layers, dims.d_model, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.d_ffn,
                        dims.page_size, num_pages, dims.rms_eps, dims.rope_base)


def make_case(dims: wl.StageDims, batch: wl.BatchSpec, seed: int = 0, num_pages: Optional[int] = None,
              mpps: Optional[int] = None, kv_fill: bool = False, init: str = "n002") -> Case:
    need = wl.pages_needed(batch, dims.page_size)
    num_pages = num_pages or need + 3
    alloc = PageAllocator(num_pages, dims.page_size)
    tables = [alloc.alloc(s, t) for s, t in enumerate(batch.total_len())]
    mpps = mpps or max(len(t) for t in tables) + 1
    bt = block_table_array(tables, mpps)
    weights_t = wl.make_weights(dims, seed, "cpu", init)
    x_t = wl.make_x(batch.n_tokens, dims.d_model, seed)
    cfg = oracle_cfg(dims, num_pages)
    if kv_fill:
        pool = wl.bf16_bits_numpy(wl.make_kv_fill(dims, num_pages, seed)).reshape(-1).copy()
    else:
        pool = np.zeros(cfg.kv_pool_elems(), dtype=np.uint16)
    return Case(dims, cfg, wl.weights_to_numpy(weights_t), weights_t, batch, bt, pool, x_t, wl.to_f32_numpy(x_t))


def rel_err(a: np.ndarray, ref: np.ndarray) -> float:
    """max |a - ref| / RMS(ref): the tolerance norm of the parity tests."""
    ref64 = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref64 ** 2)))
    return float(np.max(np.abs(np.asarray(a, dtype=np.float64) - ref64)) / max(rms, 1e-30))
