"""ctypes binding of libhorizonserve.so: the same names as the C ABI, argument marshalling only.

PyTorch appears here for what the library leaves to its caller: device memory (weights, KV pool,
workspace, inputs, outputs) and streams.  Every step of the hot path runs inside the library's CUDA
kernels; if the library is missing this module raises instead of falling back to anything.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhorizonserve.so")

HS_ABI_VERSION = 1
HS_FLAG_BF16_ACTIVATIONS = 1      # hs_stage_config_t.flags: keep h, o and act in bf16 instead of fp16
HS_FLAG_BIDIRECTIONAL = 2         # hs_stage_config_t.flags: attention without the causal mask (denoising-style block)
HS_OK, HS_ERR_INVALID_ARG, HS_ERR_INVALID_BUDGET, HS_ERR_UNSUPPORTED_SHAPE, HS_ERR_OUT_OF_PAGES, \
    HS_ERR_BAD_BLOCK_TABLE, HS_ERR_CUDA, HS_ERR_TIMEOUT, HS_ERR_NO_DEVICE, HS_ERR_UNKNOWN_SEQ = range(10)

EXPORTS = ("hs_status_str", "hs_kv_pool_bytes", "hs_workspace_bytes", "hs_stage_create", "hs_stage_destroy",
           "hs_kv_alloc", "hs_kv_free", "hs_kv_free_pages", "hs_stage_plan", "hs_stage_step", "hs_stage_status",
           "hs_stage_sm_count", "hs_op_gemm_bf16", "hs_stage_debug_buffer", "hs_stage_profile_enable",
           "hs_stage_profile_read", "hs_last_error", "hs_op_decode_attention_noalloc", "hs_op_gemm_f16",
           "hs_spatial_create", "hs_spatial_update", "hs_spatial_state", "hs_spatial_destroy",
           "hs_spatial_derive_cap", "hs_head_workspace_bytes", "hs_head_create", "hs_head_step", "hs_head_status",
           "hs_head_destroy", "hs_op_embed", "hs_temporal_create", "hs_temporal_step", "hs_temporal_destroy",
           "hs_stage_set_qkv_bias", "hs_stage_set_modulation", "hs_stage_saturation_count", "hs_op_wait_probe",
           "hs_op_decode_attention_noalloc_status", "hs_stage_plan_attention", "hs_op_gemm_split_begin")
PROFILE_CLASSES = ("rmsnorm", "gemm_qkv", "attn_prefill", "attn_decode", "attn_combine", "gemm_out", "gemm_gateup",
                   "gemm_down")


class hs_stage_config_t(C.Structure):
    _fields_ = [("abi_version", C.c_uint32), ("device", C.c_int32),
                ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ffn", C.c_int32),
                ("rms_eps", C.c_float), ("rope_base", C.c_float),
                ("page_size", C.c_int32), ("num_pages", C.c_int32), ("max_tokens", C.c_int32),
                ("max_seqs", C.c_int32), ("max_pages_per_seq", C.c_int32), ("max_position", C.c_int32),
                ("flags", C.c_uint32)]


WEIGHT_NAMES = ("g_attn", "w_q", "w_k", "w_v", "w_o", "g_mlp", "w_gate", "w_up", "w_down")


class hs_layer_weights_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES]


class hs_batch_t(C.Structure):
    _fields_ = [("n_seqs", C.c_int32), ("n_tokens", C.c_int32), ("q_len", C.c_void_p), ("ctx_len", C.c_void_p),
                ("block_tables", C.c_void_p), ("x_in", C.c_void_p), ("y_out", C.c_void_p)]


class hs_head_config_t(C.Structure):
    _fields_ = [("abi_version", C.c_uint32), ("device", C.c_int32), ("d_model", C.c_int32), ("vocab", C.c_int32),
                ("rms_eps", C.c_float), ("max_rows", C.c_int32)]


class hs_temporal_config_t(C.Structure):
    _fields_ = [("abi_version", C.c_uint32), ("n_min", C.c_int32), ("n_max", C.c_int32), ("m", C.c_int32),
                ("u_guard", C.c_double), ("long_cap", C.c_int32)]


class hs_request_view_t(C.Structure):
    _fields_ = [("id", C.c_int64), ("path", C.c_int32), ("stage", C.c_int32), ("deadline", C.c_double),
                ("remaining", C.c_double)]


class hs_spatial_config_t(C.Structure):
    _fields_ = [("abi_version", C.c_uint32), ("s_total", C.c_int32), ("s_aggr", C.c_int32), ("n_levels", C.c_int32),
                ("ladder", C.POINTER(C.c_int32)), ("b_sat", C.c_double), ("gamma", C.c_double),
                ("delta_step", C.c_int32)]


class HsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = lib().hs_last_error().decode() if status == HS_ERR_CUDA else ""
        super().__init__(f"{where}: {status_str(status)}" + (f" [{detail}]" if detail else ""))


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Loads the library (once).  Raises if it has not been built: there is no other code path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_01785_b200.build` "
                               "(the CUDA library is the only implementation)")
        l = C.CDLL(LIB_PATH)
        l.hs_status_str.restype = C.c_char_p
        l.hs_status_str.argtypes = [C.c_int]
        l.hs_kv_pool_bytes.restype = C.c_size_t
        l.hs_kv_pool_bytes.argtypes = [C.POINTER(hs_stage_config_t)]
        l.hs_workspace_bytes.restype = C.c_size_t
        l.hs_workspace_bytes.argtypes = [C.POINTER(hs_stage_config_t)]
        l.hs_stage_create.argtypes = [C.POINTER(hs_stage_config_t), C.POINTER(hs_layer_weights_t), C.c_void_p,
                                      C.c_void_p, C.POINTER(C.c_void_p)]
        l.hs_stage_destroy.argtypes = [C.c_void_p]
        l.hs_kv_alloc.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int32, C.POINTER(C.c_int32)]
        l.hs_kv_free.argtypes = [C.c_void_p, C.c_int64]
        l.hs_kv_free_pages.argtypes = [C.c_void_p]
        l.hs_kv_free_pages.restype = C.c_int32
        l.hs_stage_plan.argtypes = [C.c_void_p, C.POINTER(hs_batch_t), C.c_void_p, C.c_void_p, C.c_void_p]
        l.hs_stage_plan_attention.argtypes = [C.c_void_p, C.POINTER(hs_batch_t), C.c_void_p, C.c_int32, C.c_void_p,
                                              C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        l.hs_stage_plan_attention.restype = C.c_int
        l.hs_op_gemm_split_begin.argtypes = [C.c_int32, C.c_int32, C.c_int32]
        l.hs_op_gemm_split_begin.restype = C.c_int32
        l.hs_stage_step.argtypes = [C.c_void_p, C.POINTER(hs_batch_t), C.c_int32, C.c_void_p]
        l.hs_stage_status.argtypes = [C.c_void_p]
        l.hs_stage_sm_count.argtypes = [C.c_void_p]
        l.hs_stage_sm_count.restype = C.c_int32
        l.hs_op_gemm_bf16.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                      C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        l.hs_op_gemm_f16.argtypes = l.hs_op_gemm_bf16.argtypes
        l.hs_stage_debug_buffer.argtypes = [C.c_void_p, C.c_char_p, C.POINTER(C.c_void_p), C.POINTER(C.c_size_t)]
        l.hs_last_error.restype = C.c_char_p
        l.hs_head_workspace_bytes.restype = C.c_size_t
        l.hs_head_workspace_bytes.argtypes = [C.POINTER(hs_head_config_t)]
        l.hs_head_create.argtypes = [C.POINTER(hs_head_config_t), C.c_void_p, C.c_void_p, C.c_void_p,
                                     C.POINTER(C.c_void_p)]
        l.hs_head_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                   C.c_void_p]
        l.hs_head_status.argtypes = [C.c_void_p]
        l.hs_head_destroy.argtypes = [C.c_void_p]
        l.hs_op_embed.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32,
                                  C.c_void_p, C.c_void_p]
        l.hs_temporal_create.argtypes = [C.POINTER(hs_temporal_config_t), C.POINTER(C.c_void_p)]
        l.hs_temporal_step.argtypes = [C.c_void_p, C.c_double, C.POINTER(hs_request_view_t), C.c_int32, C.c_int32,
                                       C.POINTER(C.c_uint8), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        l.hs_temporal_destroy.argtypes = [C.c_void_p]
        l.hs_spatial_create.argtypes = [C.POINTER(hs_spatial_config_t), C.POINTER(C.c_void_p)]
        l.hs_spatial_update.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        l.hs_spatial_state.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int32)]
        l.hs_spatial_destroy.argtypes = [C.c_void_p]
        l.hs_spatial_derive_cap.argtypes = [C.POINTER(C.c_int32), C.POINTER(C.c_double), C.c_int32, C.c_int32,
                                            C.c_double, C.POINTER(C.c_int32)]
        l.hs_op_decode_attention_noalloc.argtypes = [C.c_void_p, C.c_void_p] + [C.c_int32] * 7 + \
            [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p]
        l.hs_op_decode_attention_noalloc_status.argtypes = [C.POINTER(C.c_int32)]
        l.hs_stage_saturation_count.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        l.hs_op_wait_probe.argtypes = [C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p]
        l.hs_stage_profile_enable.argtypes = [C.c_void_p, C.c_int32]
        l.hs_stage_set_qkv_bias.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        l.hs_stage_set_modulation.argtypes = [C.c_void_p, C.c_void_p]
        l.hs_stage_profile_read.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = l
    return _lib


def status_str(status: int) -> str:
    return lib().hs_status_str(int(status)).decode()


def make_config(dims, num_pages: int, max_tokens: int, max_seqs: int, max_pages_per_seq: int, max_position: int,
                device: int = 0, flags: int = 0) -> hs_stage_config_t:
    """dims: any object with n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, rms_eps, rope_base, page_size."""
    return hs_stage_config_t(HS_ABI_VERSION, device, dims.n_layers, dims.d_model, dims.n_q_heads, dims.n_kv_heads,
                             dims.head_dim, dims.d_ffn, dims.rms_eps, dims.rope_base, dims.page_size, num_pages,
                             max_tokens, max_seqs, max_pages_per_seq, max_position, flags)


def hs_kv_pool_bytes(cfg: hs_stage_config_t) -> int:
    return int(lib().hs_kv_pool_bytes(C.byref(cfg)))


def hs_workspace_bytes(cfg: hs_stage_config_t) -> int:
    return int(lib().hs_workspace_bytes(C.byref(cfg)))


def hs_stage_create(cfg: hs_stage_config_t, layer_ptrs: Optional[Sequence[Dict[str, int]]], kv_pool_ptr: int,
                    workspace_ptr: int) -> int:
    """Returns the stage handle (an integer address).  layer_ptrs: one dict of device addresses per layer."""
    arr = None
    if layer_ptrs is not None:
        arr = (hs_layer_weights_t * len(layer_ptrs))()
        for i, lw in enumerate(layer_ptrs):
            for n in WEIGHT_NAMES:
                setattr(arr[i], n, lw[n])
    out = C.c_void_p()
    st = lib().hs_stage_create(C.byref(cfg), arr, C.c_void_p(kv_pool_ptr), C.c_void_p(workspace_ptr), C.byref(out))
    if st != HS_OK:
        raise HsError(st, "hs_stage_create")
    return out.value


def hs_stage_destroy(stage: int) -> None:
    st = lib().hs_stage_destroy(C.c_void_p(stage))
    if st != HS_OK:
        raise HsError(st, "hs_stage_destroy")


def hs_kv_alloc(stage: int, seq_id: int, total_tokens: int, cap: int) -> List[int]:
    """Returns the sequence's whole block table."""
    table = (C.c_int32 * max(cap, 1))()
    n = C.c_int32(0)
    st = lib().hs_kv_alloc(C.c_void_p(stage), seq_id, total_tokens, table, cap, C.byref(n))
    if st != HS_OK:
        raise HsError(st, "hs_kv_alloc")
    return list(table[: n.value])


def hs_kv_free(stage: int, seq_id: int) -> None:
    st = lib().hs_kv_free(C.c_void_p(stage), seq_id)
    if st != HS_OK:
        raise HsError(st, "hs_kv_free")


def hs_kv_free_pages(stage: int) -> int:
    return int(lib().hs_kv_free_pages(C.c_void_p(stage)))


def hs_stage_sm_count(stage: int) -> int:
    return int(lib().hs_stage_sm_count(C.c_void_p(stage)))


class Batch:
    """Owns the host arrays of one hs_batch_t (they must stay alive across the call)."""

    def __init__(self, q_len, ctx_len, block_tables, x_in_ptr: int = 0, y_out_ptr: int = 0):
        self.q_len = np.ascontiguousarray(q_len, dtype=np.int32)
        self.ctx_len = np.ascontiguousarray(ctx_len, dtype=np.int32)
        self.block_tables = np.ascontiguousarray(block_tables, dtype=np.int32)
        self.c = hs_batch_t(len(self.q_len), int(self.q_len.sum()), self.q_len.ctypes.data, self.ctx_len.ctypes.data,
                            self.block_tables.ctypes.data, x_in_ptr, y_out_ptr)


def hs_stage_plan(stage: int, batch: Batch):
    """Returns (tok_seq, tok_pos, tok_slot) int32 arrays."""
    n = batch.c.n_tokens
    seq, pos, slot = (np.empty(max(n, 1), dtype=np.int32) for _ in range(3))
    st = lib().hs_stage_plan(C.c_void_p(stage), C.byref(batch.c), seq.ctypes.data, pos.ctypes.data, slot.ctypes.data)
    if st != HS_OK:
        raise HsError(st, "hs_stage_plan")
    return seq[:n], pos[:n], slot[:n]


def hs_stage_plan_attention(stage: int, batch: Batch, cap: int = 1 << 16):
    """Returns (decode_items [n, 8], decode_group flag, prefill_items [m, 8]) as the planner lists them."""
    dec = np.zeros((cap, 8), dtype=np.int32)
    pre = np.zeros((cap, 8), dtype=np.int32)
    n_dec, grp, n_pre = C.c_int32(0), C.c_int32(0), C.c_int32(0)
    st = lib().hs_stage_plan_attention(C.c_void_p(stage), C.byref(batch.c), dec.ctypes.data, cap, C.byref(n_dec),
                                       C.byref(grp), pre.ctypes.data, cap, C.byref(n_pre))
    if st != HS_OK:
        raise HsError(st, "hs_stage_plan_attention")
    assert n_dec.value <= cap and n_pre.value <= cap
    return dec[: n_dec.value], grp.value, pre[: n_pre.value]


def hs_op_gemm_split_begin(k_blocks: int, ks: int, i: int) -> int:
    return int(lib().hs_op_gemm_split_begin(k_blocks, ks, i))


def hs_stage_step(stage: int, batch: Batch, sm_budget: int, cuda_stream: int = 0) -> None:
    st = lib().hs_stage_step(C.c_void_p(stage), C.byref(batch.c), sm_budget, C.c_void_p(cuda_stream))
    if st != HS_OK:
        raise HsError(st, "hs_stage_step")


def hs_stage_status(stage: int) -> int:
    return int(lib().hs_stage_status(C.c_void_p(stage)))


def hs_stage_debug_buffer(stage: int, name: str):
    ptr, size = C.c_void_p(), C.c_size_t()
    st = lib().hs_stage_debug_buffer(C.c_void_p(stage), name.encode(), C.byref(ptr), C.byref(size))
    if st != HS_OK:
        raise HsError(st, "hs_stage_debug_buffer")
    return ptr.value, size.value


def hs_op_gemm_bf16(a_ptr: int, w_ptr: int, resid_ptr: int, out_ptr: int, M: int, N: int, K: int, sm_budget: int,
                    status_ptr: int, cuda_stream: int = 0, a_is_f16: bool = False) -> None:
    """out = a w^T (+ resid).  a_is_f16 selects the fp16-activation form (hs_op_gemm_f16)."""
    fn = lib().hs_op_gemm_f16 if a_is_f16 else lib().hs_op_gemm_bf16
    st = fn(C.c_void_p(a_ptr), C.c_void_p(w_ptr), C.c_void_p(resid_ptr or None), C.c_void_p(out_ptr),
                               M, N, K, sm_budget, C.c_void_p(status_ptr), C.c_void_p(cuda_stream))
    if st != HS_OK:
        raise HsError(st, "hs_op_gemm_bf16")


def hs_stage_set_qkv_bias(stage: int, layer: int, b_q: int, b_k: int, b_v: int) -> None:
    """Device pointers (0 = no bias) of the layer's q, k, v biases (bf16)."""
    st = lib().hs_stage_set_qkv_bias(C.c_void_p(stage), int(layer), C.c_void_p(b_q or None), C.c_void_p(b_k or None),
                                     C.c_void_p(b_v or None))
    if st != HS_OK:
        raise HsError(st, "hs_stage_set_qkv_bias")


def hs_stage_set_modulation(stage: int, mod: int) -> None:
    """Device pointer (0 = off) of the fp32 [n_layers, max_seqs, 6, d_model] shift / scale / gate vectors."""
    st = lib().hs_stage_set_modulation(C.c_void_p(stage), C.c_void_p(mod or None))
    if st != HS_OK:
        raise HsError(st, "hs_stage_set_modulation")


def hs_stage_profile_enable(stage: int, enable: bool) -> None:
    st = lib().hs_stage_profile_enable(C.c_void_p(stage), int(enable))
    if st != HS_OK:
        raise HsError(st, "hs_stage_profile_enable")


def hs_stage_profile_read(stage: int):
    """Returns {class name: (milliseconds, launches)} accumulated since the last read."""
    ms = np.zeros(len(PROFILE_CLASSES), dtype=np.float32)
    n = np.zeros(len(PROFILE_CLASSES), dtype=np.int32)
    st = lib().hs_stage_profile_read(C.c_void_p(stage), ms.ctypes.data, n.ctypes.data)
    if st != HS_OK:
        raise HsError(st, "hs_stage_profile_read")
    return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(PROFILE_CLASSES)}


def hs_op_decode_attention_noalloc(q_ptr: int, kv_pool_ptr: int, n_layers: int, layer: int, num_pages: int,
                                   n_q_heads: int, n_kv_heads: int, head_dim: int, kv_len, block_tables,
                                   o_ptr: int, sm_budget: int, cuda_stream: int = 0) -> None:
    """Decode attention on the library's built-in scratch area (for callers that cannot allocate device
    memory).  kv_len: int32 [n_seqs] keys per sequence; block_tables: int32 [n_seqs, max_pages_per_seq]."""
    kv_len = np.ascontiguousarray(kv_len, dtype=np.int32)
    bt = np.ascontiguousarray(block_tables, dtype=np.int32)
    st = lib().hs_op_decode_attention_noalloc(C.c_void_p(q_ptr), C.c_void_p(kv_pool_ptr), n_layers, layer, num_pages,
                                              n_q_heads, n_kv_heads, head_dim, len(kv_len), kv_len.ctypes.data,
                                              bt.ctypes.data, bt.shape[1], C.c_void_p(o_ptr), sm_budget,
                                              C.c_void_p(cuda_stream))
    if st != HS_OK:
        raise HsError(st, "hs_op_decode_attention_noalloc")


def hs_op_decode_attention_noalloc_status() -> int:
    """Device status word of the most recent hs_op_decode_attention_noalloc call (synchronise its stream first)."""
    v = C.c_int32(-1)
    st = lib().hs_op_decode_attention_noalloc_status(C.byref(v))
    if st != HS_OK:
        raise HsError(st, "hs_op_decode_attention_noalloc_status")
    return v.value


def hs_stage_saturation_count(stage: int) -> int:
    """How many fp16 activation values the stage has clamped to +-65504 since it was created."""
    v = C.c_int64(-1)
    st = lib().hs_stage_saturation_count(C.c_void_p(stage), C.byref(v))
    if st != HS_OK:
        raise HsError(st, "hs_stage_saturation_count")
    return v.value


def hs_op_wait_probe(limit_ns: int, status_ptr: int, waited_ns_ptr: int = 0, cuda_stream: int = 0) -> None:
    """Launches the bounded-wait probe: one block waits limit_ns on a barrier nobody signals, then winds down."""
    st = lib().hs_op_wait_probe(int(limit_ns), C.c_void_p(status_ptr), C.c_void_p(waited_ns_ptr or None),
                                C.c_void_p(cuda_stream))
    if st != HS_OK:
        raise HsError(st, "hs_op_wait_probe")


class SpatialController:
    """The library's spatial controller (hs_spatial_*): per step, the shared stage's SM budget from downstream
    activity and a memory-pressure sample (Sec. 4.3, Eq. 1 of the paper).  Marshalling only."""

    def __init__(self, s_total: int, s_aggr: int, ladder: Sequence[int], b_sat: float, gamma: float, delta_step: int):
        arr = (C.c_int32 * max(len(ladder), 1))(*ladder)
        cfg = hs_spatial_config_t(HS_ABI_VERSION, s_total, s_aggr, len(ladder), arr, b_sat, gamma, delta_step)
        h = C.c_void_p()
        st = lib().hs_spatial_create(C.byref(cfg), C.byref(h))
        if st != HS_OK:
            raise HsError(st, "hs_spatial_create")
        self.handle = h

    def update(self, downstream_active: bool, pressure: float):
        """Returns (s_shared, s_down) for the next step."""
        a, b = C.c_int32(), C.c_int32()
        st = lib().hs_spatial_update(self.handle, int(bool(downstream_active)), float(pressure), C.byref(a), C.byref(b))
        if st != HS_OK:
            raise HsError(st, "hs_spatial_update")
        return a.value, b.value

    def state(self):
        """(moving average of the pressure, cap in force)."""
        bhat, s = C.c_double(), C.c_int32()
        st = lib().hs_spatial_state(self.handle, C.byref(bhat), C.byref(s))
        if st != HS_OK:
            raise HsError(st, "hs_spatial_state")
        return bhat.value, s.value

    def close(self) -> None:
        if self.handle:
            lib().hs_spatial_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def hs_spatial_derive_cap(budgets: Sequence[int], latency: Sequence[float], s_total: int, tolerance: float) -> int:
    n = len(budgets)
    b = (C.c_int32 * max(n, 1))(*budgets)
    t = (C.c_double * max(n, 1))(*latency)
    out = C.c_int32()
    st = lib().hs_spatial_derive_cap(b, t, n, s_total, float(tolerance), C.byref(out))
    if st != HS_OK:
        raise HsError(st, "hs_spatial_derive_cap")
    return out.value


def make_head_config(d_model: int, vocab: int, rms_eps: float, max_rows: int, device: int = 0) -> hs_head_config_t:
    return hs_head_config_t(HS_ABI_VERSION, device, d_model, vocab, rms_eps, max_rows)


def hs_head_workspace_bytes(cfg: hs_head_config_t) -> int:
    return int(lib().hs_head_workspace_bytes(C.byref(cfg)))


def hs_head_create(cfg: hs_head_config_t, g_final_ptr: int, w_vocab_ptr: int, workspace_ptr: int) -> int:
    h = C.c_void_p()
    st = lib().hs_head_create(C.byref(cfg), C.c_void_p(g_final_ptr), C.c_void_p(w_vocab_ptr), C.c_void_p(workspace_ptr),
                              C.byref(h))
    if st != HS_OK:
        raise HsError(st, "hs_head_create")
    return h.value


def hs_head_step(head: int, y_ptr: int, rows_ptr: int, n: int, logits_ptr: int, tokens_ptr: int, sm_budget: int,
                 cuda_stream: int = 0) -> None:
    st = lib().hs_head_step(C.c_void_p(head), C.c_void_p(y_ptr), C.c_void_p(rows_ptr), n, C.c_void_p(logits_ptr),
                            C.c_void_p(tokens_ptr), sm_budget, C.c_void_p(cuda_stream))
    if st != HS_OK:
        raise HsError(st, "hs_head_step")


def hs_head_status(head: int) -> int:
    return int(lib().hs_head_status(C.c_void_p(head)))


def hs_head_destroy(head: int) -> None:
    lib().hs_head_destroy(C.c_void_p(head))


def hs_op_embed(tokens_ptr: int, n: int, table_ptr: int, vocab: int, d_model: int, x_out_ptr: int, sm_budget: int,
                status_ptr: int, cuda_stream: int = 0) -> None:
    st = lib().hs_op_embed(C.c_void_p(tokens_ptr), n, C.c_void_p(table_ptr), vocab, d_model, C.c_void_p(x_out_ptr),
                           sm_budget, C.c_void_p(status_ptr), C.c_void_p(cuda_stream))
    if st != HS_OK:
        raise HsError(st, "hs_op_embed")


class TemporalView:
    """The library's temporal scheduler view (hs_temporal_*): path rotation, slack guard, adaptive ratio and
    long-path cap of the paper (Sec. 4.2).  Marshalling only."""

    def __init__(self, n_min: int = 2, n_max: int = 8, m: int = 2, u_guard: float = 1.5, long_cap: int = 4):
        cfg = hs_temporal_config_t(HS_ABI_VERSION, n_min, n_max, m, u_guard, long_cap)
        h = C.c_void_p()
        st = lib().hs_temporal_create(C.byref(cfg), C.byref(h))
        if st != HS_OK:
            raise HsError(st, "hs_temporal_create")
        self.handle = h

    def step(self, now: float, reqs, long_admitted: int):
        """reqs: sequence of (id, path, stage, deadline, remaining).  Returns (visible flags, phase, N)."""
        n = len(reqs)
        arr = (hs_request_view_t * max(n, 1))()
        for i, (rid, path, stage, deadline, remaining) in enumerate(reqs):
            arr[i] = hs_request_view_t(rid, path, stage, deadline, remaining)
        vis = (C.c_uint8 * max(n, 1))()
        phase, ns = C.c_int32(), C.c_int32()
        st = lib().hs_temporal_step(self.handle, float(now), arr, n, long_admitted, vis, C.byref(phase), C.byref(ns))
        if st != HS_OK:
            raise HsError(st, "hs_temporal_step")
        return [bool(vis[i]) for i in range(n)], phase.value, ns.value

    def close(self) -> None:
        if self.handle:
            lib().hs_temporal_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
