"""A stage object for Python callers: torch owns the device memory and the streams, the C-ABI library
does all of the work.  This is a convenience wrapper over `binding`; it adds no computation.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import binding as B


class Stage:
    """One pipeline stage (shared backbone or downstream generator; Sec. 2.2 of the paper) on one GPU.

    weights: per layer, a dict of bf16 CUDA tensors named as in hs_layer_weights_t.
    """

    GUARD_BYTE = 0xA5

    def __init__(self, dims, weights: Sequence[Dict[str, torch.Tensor]], num_pages: int, max_tokens: int,
                 max_seqs: int, max_pages_per_seq: int, max_position: int, device: int = 0, flags: int = 0,
                 guard_bytes: int = 0):
        """guard_bytes > 0 (a multiple of 1024) puts that many bytes of a fixed pattern in front of and behind the
        workspace and the KV pool; guards_intact() tells whether anything wrote there."""
        if not torch.cuda.is_available():
            raise RuntimeError("Stage needs a CUDA device; there is no CPU implementation")
        self.dims = dims
        self.device = torch.device("cuda", device)
        self.cfg = B.make_config(dims, num_pages, max_tokens, max_seqs, max_pages_per_seq, max_position, device, flags)
        pool_bytes, ws_bytes = B.hs_kv_pool_bytes(self.cfg), B.hs_workspace_bytes(self.cfg)
        if pool_bytes == 0 or ws_bytes == 0:
            raise B.HsError(B.HS_ERR_UNSUPPORTED_SHAPE, "configuration rejected")
        self.weights = [{k: v.to(self.device, torch.bfloat16).contiguous() for k, v in lw.items()} for lw in weights]
        assert guard_bytes % 1024 == 0
        self._guarded = []
        if guard_bytes:
            def guarded(n_bytes):
                raw = torch.full((n_bytes + 2 * guard_bytes,), self.GUARD_BYTE, dtype=torch.uint8, device=self.device)
                self._guarded.append((raw, guard_bytes))
                return raw[guard_bytes: guard_bytes + n_bytes]
            self.kv_pool = guarded(pool_bytes).zero_().view(torch.bfloat16)
            self.workspace = guarded(ws_bytes)
        else:
            self.kv_pool = torch.zeros(pool_bytes // 2, dtype=torch.bfloat16, device=self.device)
            self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)
        ptrs = [{k: v.data_ptr() for k, v in lw.items()} for lw in self.weights]
        self.handle = B.hs_stage_create(self.cfg, ptrs, self.kv_pool.data_ptr(), self.workspace.data_ptr())
        self.sm_count = B.hs_stage_sm_count(self.handle)
        self.max_pages_per_seq = max_pages_per_seq

    # -- paging -----------------------------------------------------------
    def kv_alloc(self, seq_id: int, total_tokens: int) -> List[int]:
        return B.hs_kv_alloc(self.handle, seq_id, total_tokens, self.max_pages_per_seq)

    def kv_free(self, seq_id: int) -> None:
        B.hs_kv_free(self.handle, seq_id)

    def block_table_array(self, tables: Sequence[Sequence[int]]) -> np.ndarray:
        out = np.full((len(tables), self.max_pages_per_seq), -1, dtype=np.int32)
        for s, t in enumerate(tables):
            out[s, : len(t)] = t
        return out

    def kv_pool_view(self) -> torch.Tensor:
        """The pool in its interface layout [layer][K|V][page][kv_head][16][head_dim]."""
        d = self.dims
        return self.kv_pool.view(d.n_layers, 2, self.cfg.num_pages, d.n_kv_heads, d.page_size, d.head_dim)

    # -- stepping ---------------------------------------------------------
    def make_batch(self, q_len, ctx_len, block_tables, x_in: torch.Tensor, y_out: torch.Tensor) -> B.Batch:
        assert x_in.dtype == torch.bfloat16 and x_in.is_contiguous() and x_in.device == self.device
        assert y_out.dtype == torch.float32 and y_out.is_contiguous() and y_out.device == self.device
        return B.Batch(q_len, ctx_len, block_tables, x_in.data_ptr(), y_out.data_ptr())

    def step(self, batch: B.Batch, sm_budget: int, stream: Optional[torch.cuda.Stream] = None) -> None:
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        B.hs_stage_step(self.handle, batch, sm_budget, s.cuda_stream)

    def status(self) -> int:
        return B.hs_stage_status(self.handle)

    def saturation_count(self) -> int:
        """fp16 activation values clamped to +-65504 since the stage was created (0 for a well-scaled model)."""
        return B.hs_stage_saturation_count(self.handle)

    def guards_intact(self) -> bool:
        """True when the guard bytes around the workspace and the KV pool (guard_bytes of the constructor) still hold
        their pattern."""
        return all(bool((raw[:g] == self.GUARD_BYTE).all()) and bool((raw[-g:] == self.GUARD_BYTE).all())
                   for raw, g in self._guarded)

    def set_modulation(self, mod) -> None:
        """fp32 device tensor [n_layers, max_seqs, 6, d_model] (or None): per-sequence shift / scale / gate vectors
        of a conditioned block; kept alive here, read at every step."""
        assert mod is None or (mod.dtype == torch.float32 and mod.is_cuda and mod.is_contiguous() and
                               tuple(mod.shape) == (self.cfg.n_layers, self.cfg.max_seqs, 6, self.cfg.d_model))
        self._mod = mod
        B.hs_stage_set_modulation(self.handle, 0 if mod is None else mod.data_ptr())

    def set_qkv_bias(self, layer: int, b_q=None, b_k=None, b_v=None) -> None:
        """bf16 device tensors (or None) added to the layer's q, k, v projections before RoPE; kept alive here."""
        for t in (b_q, b_k, b_v):
            assert t is None or (t.dtype == torch.bfloat16 and t.is_cuda and t.is_contiguous())
        self._biases = getattr(self, "_biases", {})
        self._biases[layer] = (b_q, b_k, b_v)
        B.hs_stage_set_qkv_bias(self.handle, layer, *[0 if t is None else t.data_ptr() for t in (b_q, b_k, b_v)])

    def debug_tensor(self, name: str) -> torch.Tensor:
        """Copy of a private intermediate, shaped [max_tokens, width] ("q" is bf16; "h", "o" and "act" are
        fp16, or bf16 when the stage was made with HS_FLAG_BF16_ACTIVATIONS), or of the SM census ("smid";
        int32 [kernel class, block]; the first request switches the census on)."""
        ptr, size = B.hs_stage_debug_buffer(self.handle, name)
        off = ptr - self.workspace.data_ptr()
        raw = self.workspace[off: off + size].clone()
        if name == "smid":
            return raw.view(torch.int32).view(len(B.PROFILE_CLASSES), -1)
        bf16 = name == "q" or (self.cfg.flags & B.HS_FLAG_BF16_ACTIVATIONS)
        return raw.view(torch.bfloat16 if bf16 else torch.float16).view(self.cfg.max_tokens, -1)

    def close(self) -> None:
        if self.handle:
            B.hs_stage_destroy(self.handle)
            self.handle = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
