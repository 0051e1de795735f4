"""Set-up shared by the GPU parity tests: runs a Case (see helpers.py) through the C-ABI library."""
from __future__ import annotations

from typing import Optional

import numpy as np
import torch

from paper_2608_01785_b200 import workloads as wl
from paper_2608_01785_b200.stage import Stage
from tests.helpers import Case


def make_stage(case: Case, max_tokens: Optional[int] = None, max_position: Optional[int] = None,
               weights=None, flags: int = 0, guard_bytes: int = 0) -> Stage:
    """A stage with the case's dims and weights whose pool starts as a copy of the case's pool and whose
    allocator has handed out the case's block tables (the library's allocator must reproduce them)."""
    batch = case.batch
    st = Stage(case.dims, weights if weights is not None else case.weights_t, case.cfg.num_pages,
               max_tokens or batch.n_tokens, batch.n_seqs, case.mpps, max_position or max(batch.total_len()),
               flags=flags, guard_bytes=guard_bytes)
    st.kv_pool.copy_(wl.bits_to_bf16_tensor(case.kv_pool, st.device))
    tables = [st.kv_alloc(s, t) for s, t in enumerate(batch.total_len())]
    bt = st.block_table_array(tables)
    assert np.array_equal(bt, case.block_tables), "library allocator disagrees with the oracle's"
    return st


def run_step(st: Stage, case: Case, budget: int, q_len=None, ctx_len=None, x_t=None, block_tables=None,
             stream=None, expect_saturation: bool = False):
    """One hs_stage_step; returns (y float32 numpy [T, d], pool uint16 numpy, flat)."""
    q_len = case.batch.q_len if q_len is None else q_len
    ctx_len = case.batch.ctx_len if ctx_len is None else ctx_len
    x = (case.x_t if x_t is None else x_t).to(st.device).contiguous()
    y = torch.full((x.shape[0], case.dims.d_model), float("nan"), device=st.device)
    b = st.make_batch(q_len, ctx_len, case.block_tables if block_tables is None else block_tables, x, y)
    st.step(b, budget, stream)
    torch.cuda.synchronize()
    assert st.status() == 0
    if not expect_saturation:
        assert st.saturation_count() == 0, "a regular case clamped fp16 activations"
    return y.cpu().numpy(), wl.bf16_bits_numpy(st.kv_pool).reshape(-1)


def bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)
