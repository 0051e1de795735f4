"""ctypes front end of the CPU oracle (hs_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product path never imports this package.

Two builds of the same C file exist: float32 (the oracle proper) and float64
(used to bound the oracle's own rounding).  Tensors cross as numpy arrays;
weights and activations carry values that were already rounded to bf16 by the
input generator and are widened exactly.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hs_oracle.c")
_LIBS: Dict[str, C.CDLL] = {}

ROUND_H, ROUND_Q, ROUND_P, ROUND_O, ROUND_ACT = 1, 2, 4, 8, 16
ROUND_ALL = 31
ROUND_ACT_F16 = 32          # with ROUND_H / ROUND_O / ROUND_ACT: those three go to fp16 instead of bf16


def lib_path(precision: str) -> str:
    return os.path.join(_HERE, f"libhs_oracle_{precision}.so")


def build(force: bool = False) -> None:
    """Compile both precisions of the oracle with gcc (AVX2 baseline, OpenMP)."""
    for precision, real in (("f32", "float"), ("f64", "double")):
        out = lib_path(precision)
        if not force and os.path.exists(out) and os.path.getmtime(out) >= os.path.getmtime(_SRC):
            continue
        cmd = ["gcc", "-O3", "-march=x86-64-v3", "-fopenmp", "-fPIC", "-shared", "-std=c11",
               f"-DHSO_REAL={real}", _SRC, "-o", out, "-lm"]
        subprocess.run(cmd, check=True)


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim",
                                          "d_ffn", "page_size", "num_pages")] + \
               [("rms_eps", C.c_float), ("rope_base", C.c_float), ("bidirectional", C.c_int32)]


class _Layer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("g_attn", "w_q", "w_k", "w_v", "w_o", "g_mlp", "w_gate", "w_up",
                                           "w_down", "b_q", "b_k", "b_v", "mod")]


WEIGHT_NAMES = ("g_attn", "w_q", "w_k", "w_v", "w_o", "g_mlp", "w_gate", "w_up", "w_down")
# optional entries of a layer's dict: biases of the q, k, v projections; "mod" [n_seqs, 6, d]: per-sequence
# shift / scale / gate vectors of a conditioned (adaLN-Zero) block for the attention and the MLP branch
BIAS_NAMES = ("b_q", "b_k", "b_v", "mod")


def _load(precision: str) -> C.CDLL:
    if precision not in _LIBS:
        build()
        lib = C.CDLL(lib_path(precision))
        lib.hso_bf16_rne.restype = C.c_uint16
        lib.hso_bf16_rne.argtypes = [C.c_float]
        lib.hso_bf16_to_float.restype = C.c_float
        lib.hso_bf16_to_float.argtypes = [C.c_uint16]
        lib.hso_silu_f32.restype = C.c_float
        lib.hso_silu_f32.argtypes = [C.c_float]
        lib.hso_kv_pool_elems.restype = C.c_size_t
        lib.hso_sizeof_real.restype = C.c_int
        _LIBS[precision] = lib
    return _LIBS[precision]


@dataclass
class OracleConfig:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    page_size: int
    num_pages: int
    rms_eps: float = 1e-6
    rope_base: float = 10000.0
    bidirectional: bool = False      # no causal mask: every token sees all keys of its sequence

    def c(self) -> _Cfg:
        return _Cfg(self.n_layers, self.d_model, self.n_q_heads, self.n_kv_heads, self.head_dim, self.d_ffn,
                    self.page_size, self.num_pages, self.rms_eps, self.rope_base, int(self.bidirectional))

    def kv_pool_elems(self) -> int:
        return self.n_layers * 2 * self.num_pages * self.n_kv_heads * self.page_size * self.head_dim


def _ptr(a: np.ndarray) -> C.c_void_p:
    return C.c_void_p(a.ctypes.data)


class Oracle:
    """One precision of the oracle ("f32" is the reference, "f64" its check)."""

    def __init__(self, precision: str = "f32"):
        assert precision in ("f32", "f64")
        self.lib = _load(precision)
        self.dtype = np.float32 if precision == "f32" else np.float64
        assert self.lib.hso_sizeof_real() == np.dtype(self.dtype).itemsize

    # -- scalar helpers ---------------------------------------------------
    def bf16_rne(self, f: float) -> int:
        return int(self.lib.hso_bf16_rne(C.c_float(f)))

    def bf16_to_float(self, bits: int) -> float:
        return float(self.lib.hso_bf16_to_float(C.c_uint16(bits)))

    def silu(self, z: float) -> float:
        return float(self.lib.hso_silu_f32(C.c_float(z)))

    def set_operand_rounding(self, mask: int) -> None:
        self.lib.hso_set_operand_rounding(C.c_int(mask))

    # -- array helpers ----------------------------------------------------
    def _arr(self, a) -> np.ndarray:
        return np.ascontiguousarray(np.asarray(a), dtype=self.dtype)

    def rmsnorm(self, x, g, eps: float) -> np.ndarray:
        x, g = self._arr(x), self._arr(g)
        T, d = x.shape
        h = np.empty_like(x)
        self.lib.hso_rmsnorm(C.c_int(T), C.c_int(d), _ptr(x), _ptr(g), C.c_float(eps), _ptr(h))
        return h

    def linear(self, a, w) -> np.ndarray:
        a, w = self._arr(a), self._arr(w)
        T, K = a.shape
        N, K2 = w.shape
        assert K == K2
        y = np.empty((T, N), dtype=self.dtype)
        self.lib.hso_linear(C.c_int(T), C.c_int(N), C.c_int(K), _ptr(a), _ptr(w), _ptr(y))
        return y

    def rope(self, z, pos: int, base: float) -> np.ndarray:
        """z: [n_heads, Dh] of one token; returns the rotated copy."""
        z = self._arr(z).copy()
        n_heads, Dh = z.shape
        self.lib.hso_rope(C.c_int(n_heads), C.c_int(Dh), C.c_int(pos), C.c_float(base), _ptr(z))
        return z

    def attend(self, cfg: OracleConfig, kv_pool: np.ndarray, layer: int, table_row, pos: int, hq: int, q):
        """Returns (o[Dh], probs[pos+1]) of one query vector."""
        assert kv_pool.dtype == np.uint16 and kv_pool.size == cfg.kv_pool_elems()
        q = self._arr(q)
        row = np.ascontiguousarray(table_row, dtype=np.int32)
        o = np.empty(cfg.head_dim, dtype=self.dtype)
        probs = np.empty(pos + 1, dtype=self.dtype)
        c = cfg.c()
        self.lib.hso_attend(C.byref(c), _ptr(kv_pool), C.c_int(layer), _ptr(row), C.c_int(pos), C.c_int(hq),
                            _ptr(q), _ptr(o), _ptr(probs))
        return o, probs

    def _layers(self, weights: Sequence[Dict[str, np.ndarray]]):
        keep: List[np.ndarray] = []
        arr = (_Layer * len(weights))()
        for i, lw in enumerate(weights):
            for name in WEIGHT_NAMES:
                a = self._arr(lw[name])
                keep.append(a)
                setattr(arr[i], name, a.ctypes.data)
            for name in BIAS_NAMES:
                if lw.get(name) is not None:
                    a = self._arr(lw[name])
                    keep.append(a)
                    setattr(arr[i], name, a.ctypes.data)
        return arr, keep

    def layer(self, cfg: OracleConfig, layer_weights: Dict[str, np.ndarray], layer: int, kv_pool: np.ndarray,
              q_len, ctx_len, block_tables, x, row_mask: Optional[np.ndarray] = None,
              want_kv_pre: bool = False):
        """Runs one layer; returns (x_out, kv_pre or None).  kv_pool is updated in place."""
        assert kv_pool.dtype == np.uint16 and kv_pool.flags.c_contiguous and kv_pool.size == cfg.kv_pool_elems()
        q_len = np.ascontiguousarray(q_len, dtype=np.int32)
        ctx_len = np.ascontiguousarray(ctx_len, dtype=np.int32)
        bt = np.ascontiguousarray(block_tables, dtype=np.int32)
        n_seqs, mpps = bt.shape
        x = self._arr(x).copy()
        T = int(q_len.sum())
        assert x.shape == (T, cfg.d_model)
        arr, keep = self._layers([layer_weights])
        mask = None if row_mask is None else np.ascontiguousarray(row_mask, dtype=np.uint8)
        kv_pre = np.empty((T, 2, cfg.n_kv_heads * cfg.head_dim), dtype=self.dtype) if want_kv_pre else None
        c = cfg.c()
        rc = self.lib.hso_layer(C.byref(c), arr, C.c_int(layer), _ptr(kv_pool), C.c_int(n_seqs), _ptr(q_len),
                                _ptr(ctx_len), _ptr(bt), C.c_int(mpps), _ptr(x),
                                _ptr(mask) if mask is not None else None,
                                _ptr(kv_pre) if kv_pre is not None else None)
        if rc != 0:
            raise ValueError("oracle: malformed batch")
        del keep
        return x, kv_pre

    def step(self, cfg: OracleConfig, weights: Sequence[Dict[str, np.ndarray]], kv_pool: np.ndarray, q_len,
             ctx_len, block_tables, x_in, last_layer_row_mask: Optional[np.ndarray] = None) -> np.ndarray:
        """Runs all layers; returns y[T,d].  kv_pool (uint16 bf16 bits) is updated in place."""
        assert kv_pool.dtype == np.uint16 and kv_pool.flags.c_contiguous and kv_pool.size == cfg.kv_pool_elems()
        assert len(weights) == cfg.n_layers
        q_len = np.ascontiguousarray(q_len, dtype=np.int32)
        ctx_len = np.ascontiguousarray(ctx_len, dtype=np.int32)
        bt = np.ascontiguousarray(block_tables, dtype=np.int32)
        n_seqs, mpps = bt.shape
        x_in = self._arr(x_in)
        T = int(q_len.sum())
        assert x_in.shape == (T, cfg.d_model)
        y = np.empty_like(x_in)
        arr, keep = self._layers(weights)
        mask = None if last_layer_row_mask is None else np.ascontiguousarray(last_layer_row_mask, dtype=np.uint8)
        c = cfg.c()
        rc = self.lib.hso_step(C.byref(c), arr, _ptr(kv_pool), C.c_int(n_seqs), _ptr(q_len), _ptr(ctx_len),
                               _ptr(bt), C.c_int(mpps), _ptr(x_in), _ptr(y),
                               _ptr(mask) if mask is not None else None)
        if rc != 0:
            raise ValueError("oracle: malformed batch")
        del keep
        return y
