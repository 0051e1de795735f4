"""Seeded synthetic inputs shaped like the paper's omni-serving workloads.

This module only draws numbers and lengths; it contains none of the step's
arithmetic and is the one module that both the CUDA path's callers and the CPU
oracle's tests use, so that both sides receive the same buffers.

Stand-in for: the evaluated pipelines (a 7B-class shared backbone with a small
talker decoder behind it, Sec. 6.1) driven by mixed text / speech / image
request streams.  Model weights and datasets are not available, so only their
shapes are kept: layer dimensions, prompt-chunk and KV lengths, class mix.

Every float tensor is drawn in float32 and rounded once to bf16
(round-to-nearest-even); sub-streams (weights / activations / lengths / cache
fill / trace) are spawned from the seed so that changing the batch does not
change the weights.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

WEIGHT_NAMES = ("g_attn", "w_q", "w_k", "w_v", "w_o", "g_mlp", "w_gate", "w_up", "w_down")
_STREAM = {"weights": 1, "x": 2, "lengths": 3, "kv": 4, "trace": 5, "policy": 6, "modulation": 7}


@dataclass(frozen=True)
class StageDims:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    rms_eps: float = 1e-6
    rope_base: float = 10000.0
    page_size: int = 16

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def params_per_layer(self) -> int:
        d = self.d_model
        return d * (self.q_dim + 2 * self.kv_dim) + d * self.q_dim + 3 * d * self.d_ffn

    def weight_shapes(self) -> Dict[str, Tuple[int, ...]]:
        d, F = self.d_model, self.d_ffn
        return {"g_attn": (d,), "w_q": (self.q_dim, d), "w_k": (self.kv_dim, d), "w_v": (self.kv_dim, d),
                "w_o": (d, self.q_dim), "g_mlp": (d,), "w_gate": (F, d), "w_up": (F, d), "w_down": (d, F)}


DIMS = {
    "c1_tiny": StageDims(1, 256, 4, 2, 64, 688),
    "c2_shared": StageDims(4, 2048, 16, 2, 128, 5632),
    "c3_7b": StageDims(28, 3584, 28, 4, 128, 18944),
    "c4_talker": StageDims(12, 1024, 16, 4, 64, 2816),
}
DIMS["c3_decode"] = DIMS["c3_7b"]
# A denoising-style (DiT-like) downstream stage, the visual generator kind of the paper's Sec. 2.1: the talker's
# width and depth with multi-head attention, no causal mask and per-image shift / scale / gate conditioning; a step
# denoises 4 images of 256 latent tokens.
DIMS["c6_dit"] = StageDims(12, 1024, 16, 16, 64, 2816)
STAGE_FLAGS = {"c6_dit": 2}      # hs_stage_config_t.flags by workload (2 = no causal mask)
CONDITIONED = {"c6_dit"}         # workloads whose stage runs with per-sequence shift / scale / gate vectors
SM_BUDGETS = {
    "c1_tiny": (148, 8),
    "c2_shared": (148, 112, 74, 37),
    "c3_7b": (148, 120, 96, 74, 48),
    "c4_corun": (120, 96, 74),
}


@dataclass
class BatchSpec:
    """Sequences of one step, prefill chunks first then decodes (one new token each)."""
    q_len: List[int]
    ctx_len: List[int]

    @property
    def n_seqs(self) -> int:
        return len(self.q_len)

    @property
    def n_tokens(self) -> int:
        return int(sum(self.q_len))

    def total_len(self) -> List[int]:
        return [q + c for q, c in zip(self.q_len, self.ctx_len)]


def _subseed(seed: int, stream: str, index: int = 0) -> int:
    return int(np.random.SeedSequence([seed, _STREAM[stream], index]).generate_state(1, dtype=np.uint64)[0] >> 1)


def _rng(seed: int, stream: str, index: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(_subseed(seed, stream, index)))


def make_batch(name: str, seed: int) -> BatchSpec:
    """Batch structure of a named configuration (lengths only)."""
    r = _rng(seed, "lengths")
    if name == "c1_tiny":
        return BatchSpec([32, 48, 1, 1], [0, 0, 40, 64])
    if name == "c2_shared":
        pre = r.integers(128, 1025, size=8).tolist()
        dec = r.integers(256, 2049, size=32).tolist()
        return BatchSpec(pre + [1] * 32, [0] * 8 + dec)
    if name == "c3_7b":
        dec = r.integers(512, 4097, size=64).tolist()
        return BatchSpec([2048] + [1] * 64, [0] + dec)
    if name == "c3_decode":          # config 3 without its prefill chunk: a decode-only tick of the trace replay
        dec = r.integers(512, 4097, size=64).tolist()
        return BatchSpec([1] * 64, dec)
    if name == "c4_talker":
        dec = r.integers(128, 1025, size=16).tolist()
        return BatchSpec([1] * 16, dec)
    if name == "c6_dit":
        return BatchSpec([256] * 4, [0] * 4)
    raise KeyError(name)


def _normal_bf16(shape, std: float, mean: float, gen: torch.Generator, device) -> torch.Tensor:
    t = torch.empty(shape, dtype=torch.float32, device=device)
    t.normal_(mean, std, generator=gen)
    return t.to(torch.bfloat16)


def make_layer_weights(dims: StageDims, seed: int, layer: int, device="cpu",
                       init: str = "n002") -> Dict[str, torch.Tensor]:
    """bf16 weights of one layer: matrices ~ N(0, 0.02), gains ~ 1 + 0.02 N(0,1).
    init="depth_scaled" draws w_o and w_down with std 0.02 / sqrt(2 L)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(_subseed(seed, "weights", layer))
    out = {}
    for name, shape in dims.weight_shapes().items():
        if name.startswith("g_"):
            out[name] = _normal_bf16(shape, 0.02, 1.0, gen, device)
        else:
            std = 0.02
            if init == "depth_scaled" and name in ("w_o", "w_down"):
                std = 0.02 / float(np.sqrt(2.0 * dims.n_layers))
            out[name] = _normal_bf16(shape, std, 0.0, gen, device)
    return out


def make_weights(dims: StageDims, seed: int, device="cpu", init: str = "n002") -> List[Dict[str, torch.Tensor]]:
    return [make_layer_weights(dims, seed, l, device, init) for l in range(dims.n_layers)]


def make_x(n_tokens: int, d_model: int, seed: int, device="cpu", index: int = 0) -> torch.Tensor:
    """Input hidden states ~ N(0,1), bf16 [n_tokens, d_model]."""
    gen = torch.Generator(device=device)
    gen.manual_seed(_subseed(seed, "x", index))
    return _normal_bf16((n_tokens, d_model), 1.0, 0.0, gen, device)


def make_modulation(dims: StageDims, n_seqs: int, seed: int, device="cpu") -> torch.Tensor:
    """Shift / scale / gate vectors of a conditioned block, fp32 [n_layers, n_seqs, 6, d_model]: shift and scale
    ~ N(0, 0.1), gates ~ N(1, 0.1) (the magnitudes of a trained conditioning path are not public; these keep the
    residual stream's scale)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(_subseed(seed, "modulation", 0))
    m = torch.empty((dims.n_layers, n_seqs, 6, dims.d_model), dtype=torch.float32, device=device)
    m.normal_(0.0, 0.1, generator=gen)
    m[:, :, 2] += 1.0
    m[:, :, 5] += 1.0
    return m


def kv_pool_shape(dims: StageDims, num_pages: int) -> Tuple[int, ...]:
    """[layer][K or V][page][kv_head][slot][head_dim] -- the interface layout of the cache."""
    return (dims.n_layers, 2, num_pages, dims.n_kv_heads, dims.page_size, dims.head_dim)


def make_kv_fill(dims: StageDims, num_pages: int, seed: int, device="cpu") -> torch.Tensor:
    """A pool filled with bf16 N(0,1) values: stands in for context written by earlier steps
    where replaying those steps in the oracle would take too long."""
    gen = torch.Generator(device=device)
    gen.manual_seed(_subseed(seed, "kv"))
    return _normal_bf16(kv_pool_shape(dims, num_pages), 1.0, 0.0, gen, device)


def make_kv_fill_layer(dims: StageDims, num_pages: int, seed: int, layer: int, device="cpu") -> torch.Tensor:
    """One layer's [K or V][page][kv_head][slot][head_dim] block of such a fill, from a sub-stream of its own, for
    stages too deep to draw the whole pool at once."""
    gen = torch.Generator(device=device)
    gen.manual_seed(_subseed(seed, "kv", layer + 1))
    return _normal_bf16(kv_pool_shape(dims, num_pages)[1:], 1.0, 0.0, gen, device)


def pages_needed(batch: BatchSpec, page_size: int = 16) -> int:
    return int(sum(-(-t // page_size) for t in batch.total_len()))


# --- numpy views for the oracle --------------------------------------------
def to_f32_numpy(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float32).numpy()


def bf16_bits_numpy(t: torch.Tensor) -> np.ndarray:
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16_tensor(bits: np.ndarray, device="cpu") -> torch.Tensor:
    assert bits.dtype == np.uint16
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(device)


def weights_to_numpy(weights: List[Dict[str, torch.Tensor]]) -> List[Dict[str, np.ndarray]]:
    return [{k: to_f32_numpy(v) for k, v in lw.items()} for lw in weights]


# --- downstream-heavy request trace ----------------------------------------
@dataclass
class Request:
    rid: int
    arrival_s: float
    out_class: str            # "text" | "speech" | "image"
    prompt_len: int
    backbone_out: int         # backbone decode tokens
    talker_out: int           # downstream (talker-shaped) tokens; 0 for text


def make_trace(rate_per_s: float, n_requests: int = 2000, seed: int = 4) -> List[Request]:
    """Poisson arrivals; classes text/speech/image 30/50/20; prompt lengths lognormal
    (median 600, sigma 0.6, clipped 64..4096); text outputs 64..512 backbone tokens;
    long-path requests add 200..1500 downstream tokens."""
    r = _rng(seed, "trace", int(rate_per_s * 1000))
    t = 0.0
    out = []
    for i in range(n_requests):
        t += float(r.exponential(1.0 / rate_per_s))
        cls = ("text", "speech", "image")[int(r.choice(3, p=[0.3, 0.5, 0.2]))]
        prompt = int(np.clip(np.rint(np.exp(r.normal(np.log(600.0), 0.6))), 64, 4096))
        backbone_out = int(r.integers(64, 513))
        talker_out = 0 if cls == "text" else int(r.integers(200, 1501))
        out.append(Request(i, t, cls, prompt, backbone_out, talker_out))
    return out
