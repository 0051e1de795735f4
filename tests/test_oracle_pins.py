"""Pins of the CPU oracle against things other than itself: closed forms,
invariants, brute force on tiny inputs, and float64 library routines.

Each test is chosen so that one plausible mistake in hs_oracle.c (a dropped
term, a wrong index or sign, a transposed operand, an off-by-one in the causal
bound or in the page arithmetic) fails it.
"""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle.oracle import Oracle, OracleConfig
from oracle.paging import PageAllocator, block_table_array
from paper_2608_01785_b200 import workloads as wl
from tests.helpers import make_case, oracle_cfg, rel_err

TINY = wl.DIMS["c1_tiny"]


# ------------------------------------------------------------------ bf16 --
def test_bf16_rne_matches_library_rounding(oracle32):
    g = torch.Generator().manual_seed(1)
    vals = torch.randn(4096, generator=g) * torch.logspace(-6, 6, 4096)
    # exact ties: 1 + 2^-8 (ties to even -> 1.0), 1 + 3*2^-8 (-> 1 + 2^-6)
    vals = torch.cat([vals, torch.tensor([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -1.0 - 2 ** -8, 0.0, 65280.0])])
    want = vals.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle32.bf16_rne(float(v)) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, want)
    assert oracle32.bf16_to_float(oracle32.bf16_rne(1.0 + 2 ** -8)) == 1.0
    assert oracle32.bf16_to_float(oracle32.bf16_rne(1.0 + 3 * 2 ** -8)) == 1.0 + 2 ** -6


# ---------------------------------------------------------------- linear --
def test_linear_is_a_times_w_transposed(oracle32, oracle64):
    r = np.random.default_rng(0)
    a = r.standard_normal((19, 70))
    w = r.standard_normal((33, 70))          # [out, in]
    want = a @ w.T
    assert np.allclose(oracle64.linear(a, w), want, rtol=0, atol=1e-12)
    assert rel_err(oracle32.linear(a, w), want) < 1e-5
    # a transposed-operand mistake cannot survive a non-square one-hot probe
    e = np.zeros((1, 70)); e[0, 3] = 1.0
    assert np.allclose(oracle64.linear(e, w)[0], w[:, 3])


# --------------------------------------------------------------- RMSNorm --
def test_rmsnorm_unit_rms_and_scale_invariance(oracle64):
    r = np.random.default_rng(1)
    x = r.standard_normal((5, 256)) * 3.0
    h = oracle64.rmsnorm(x, np.ones(256), 0.0)
    assert np.allclose(np.sqrt((h ** 2).mean(axis=1)), 1.0, atol=1e-12)
    g = 1.0 + 0.1 * r.standard_normal(256)
    h1 = oracle64.rmsnorm(x, g, 0.0)
    h2 = oracle64.rmsnorm(7.5 * x, g, 0.0)
    assert np.allclose(h1, h2, atol=1e-12)
    assert np.allclose(h1, h * g, atol=1e-12)            # the gain multiplies per column
    # eps sits inside the root, added to the mean of squares: x = 0 row, and a closed form
    x1 = np.full((1, 4), 2.0)
    assert np.allclose(oracle64.rmsnorm(x1, np.ones(4), 5.0), 2.0 / 3.0, atol=1e-12)


def test_rmsnorm_factors_out_of_the_projection_behind_it(oracle64):
    """rmsnorm(x) W^T = diag(r) ((x o g) W^T) with r = 1 / sqrt(mean(x^2) + eps): the identity behind folding the norm
    into the GEMMs around it (the 16-bit rounding then falls on x o g instead of on r (x o g))."""
    r = np.random.default_rng(17)
    x = r.standard_normal((9, 160)) * np.array([0.01, 0.3, 1, 2, 5, 10, 40, 100, 1000])[:, None]
    g = 1.0 + 0.3 * r.standard_normal(160)
    w = r.standard_normal((48, 160)) / math.sqrt(160)
    eps = float(np.float32(1e-6))                        # the oracle takes eps as a C float
    rs = 1.0 / np.sqrt((x ** 2).mean(axis=1) + eps)
    before = oracle64.linear(oracle64.rmsnorm(x, g, eps), w)
    after = rs[:, None] * oracle64.linear(x * g, w)
    assert np.allclose(before, after, rtol=1e-12, atol=1e-12)
    # a mistake in the factor (eps outside the root, the mean over the wrong axis, g left out) does not survive
    assert not np.allclose(before, (1.0 / (np.sqrt((x ** 2).mean(axis=1)) + eps))[:, None] * oracle64.linear(x * g, w), rtol=1e-9, atol=0)
    assert not np.allclose(before, rs[:, None] * oracle64.linear(x, w), rtol=1e-3, atol=1e-6)


def test_rmsnorm_matches_library(oracle32):
    r = np.random.default_rng(2)
    x = r.standard_normal((7, 96)).astype(np.float32)
    g = (1 + 0.02 * r.standard_normal(96)).astype(np.float32)
    want = F.rms_norm(torch.from_numpy(x).double(), (96,), torch.from_numpy(g).double(), 1e-6).numpy()
    assert rel_err(oracle32.rmsnorm(x, g, 1e-6), want) < 1e-6


# ------------------------------------------------------------------ RoPE --
def test_rope_identity_norm_and_pairing(oracle64):
    r = np.random.default_rng(3)
    z = r.standard_normal((3, 64))
    assert np.array_equal(oracle64.rope(z, 0, 10000.0), z)
    for pos in (1, 17, 4095):
        zr = oracle64.rope(z, pos, 10000.0)
        # every (i, i+Dh/2) pair keeps its norm
        n0 = z[:, :32] ** 2 + z[:, 32:] ** 2
        n1 = zr[:, :32] ** 2 + zr[:, 32:] ** 2
        assert np.allclose(n0, n1, rtol=1e-12)
    # closed form: pair 0 has theta = 1, so position p rotates (1, 0) to (cos p, sin p);
    # the last pair has theta = base^(-(Dh-2)/Dh)
    e = np.zeros((1, 64)); e[0, 0] = 1.0; e[0, 31] = 1.0
    zr = oracle64.rope(e, 5, 10000.0)[0]
    assert math.isclose(zr[0], math.cos(5.0), abs_tol=1e-12) and math.isclose(zr[32], math.sin(5.0), abs_tol=1e-12)
    th = 10000.0 ** (-62.0 / 64.0)
    assert math.isclose(zr[31], math.cos(5 * th), abs_tol=1e-12) and math.isclose(zr[63], math.sin(5 * th), abs_tol=1e-12)


def test_rope_relative_position_property(oracle64):
    r = np.random.default_rng(4)
    q = r.standard_normal((1, 128)); k = r.standard_normal((1, 128))
    base = 10000.0
    s0 = float(oracle64.rope(q, 9, base)[0] @ oracle64.rope(k, 4, base)[0])
    s1 = float(oracle64.rope(q, 1009, base)[0] @ oracle64.rope(k, 1004, base)[0])
    assert abs(s0 - s1) < 1e-9
    # complex-multiplication form of the same rotation (independent formulation)
    half = 64
    zc = torch.complex(torch.from_numpy(q[0, :half]), torch.from_numpy(q[0, half:]))
    ang = 9.0 * torch.pow(torch.tensor(base, dtype=torch.float64), -torch.arange(half, dtype=torch.float64) * 2 / 128)
    rot = zc * torch.polar(torch.ones(half, dtype=torch.float64), ang)
    want = torch.cat([rot.real, rot.imag]).numpy()
    assert np.allclose(oracle64.rope(q, 9, base)[0], want, atol=1e-12)


# ------------------------------------------------------------------ SiLU --
def test_silu_closed_forms(oracle32):
    assert oracle32.silu(0.0) == 0.0
    assert math.isclose(oracle32.silu(30.0), 30.0, rel_tol=1e-6)
    assert abs(oracle32.silu(-30.0)) < 1e-10
    for z in (0.3, 1.7, 5.0):
        assert math.isclose(oracle32.silu(z) - oracle32.silu(-z), z, rel_tol=1e-6)
    assert math.isclose(oracle32.silu(1.0), 1.0 / (1.0 + math.exp(-1.0)), rel_tol=1e-6)


# ------------------------------------------------------------- attention --
def _single_seq_cache(orc, n_tokens, Hkv, Dh, K, V, page_size=16, perm=None):
    """Places K,V [n, Hkv, Dh] (float, exactly bf16-representable) in a 1-layer paged pool."""
    n_pages = -(-n_tokens // page_size)
    pages = list(range(n_pages)) if perm is None else list(perm[:n_pages])
    num_pages = max(pages) + 2
    cfg = OracleConfig(1, 8, Hkv, Hkv, Dh, 8, page_size, num_pages)
    pool = np.full((1, 2, num_pages, Hkv, page_size, Dh), 0x7fc0, dtype=np.uint16)   # NaN canary
    kb = wl.bf16_bits_numpy(torch.from_numpy(K).to(torch.bfloat16))
    vb = wl.bf16_bits_numpy(torch.from_numpy(V).to(torch.bfloat16))
    for j in range(n_tokens):
        pool[0, 0, pages[j // page_size], :, j % page_size, :] = kb[j]
        pool[0, 1, pages[j // page_size], :, j % page_size, :] = vb[j]
    return cfg, pool.reshape(-1), np.asarray(pages, dtype=np.int32)


def _bf16_exact(a):
    return torch.from_numpy(a).to(torch.bfloat16).double().numpy()


def test_softmax_rows_sum_to_one_and_shift_invariance(oracle32, oracle64):
    r = np.random.default_rng(5)
    n, Dh = 37, 64
    K = _bf16_exact(r.standard_normal((n, 1, Dh))); V = _bf16_exact(r.standard_normal((n, 1, Dh)))
    K[:, 0, Dh - 1] = 0.0
    q = r.standard_normal(Dh); q[Dh - 1] = 1.0
    for orc, tol in ((oracle32, 1e-6), (oracle64, 1e-14)):
        cfg, pool, pages = _single_seq_cache(orc, n, 1, Dh, K, V)
        o0, p0 = orc.attend(cfg, pool, 0, pages, n - 1, 0, q)
        assert abs(float(p0.sum()) - 1.0) <= tol
        assert np.all(p0 > 0)
        # adding a constant to every score (last key channel = c, last q channel = 1) changes nothing
        K2 = K.copy(); K2[:, 0, Dh - 1] = 48.0
        cfg, pool2, pages = _single_seq_cache(orc, n, 1, Dh, K2, V)
        o1, p1 = orc.attend(cfg, pool2, 0, pages, n - 1, 0, q)
        assert np.allclose(p0, p1, atol=20 * tol) and np.allclose(o0, o1, atol=100 * tol)


def test_attention_closed_forms(oracle64):
    r = np.random.default_rng(6)
    Dh, n = 64, 21
    K = _bf16_exact(r.standard_normal((n, 1, Dh)))
    v0 = _bf16_exact(r.standard_normal(Dh))
    # constant V -> output is V
    cfg, pool, pages = _single_seq_cache(oracle64, n, 1, Dh, K, np.tile(v0, (n, 1, 1)))
    o, _ = oracle64.attend(cfg, pool, 0, pages, n - 1, 0, r.standard_normal(Dh))
    assert np.allclose(o, v0, atol=1e-12)
    # single key -> o = v of that key, whatever q
    V = _bf16_exact(r.standard_normal((n, 1, Dh)))
    cfg, pool, pages = _single_seq_cache(oracle64, n, 1, Dh, K, V)
    o, p = oracle64.attend(cfg, pool, 0, pages, 0, 0, r.standard_normal(Dh))
    assert np.allclose(o, V[0, 0], atol=1e-12) and p.shape == (1,)
    # q = 0 -> equal scores -> arithmetic mean over keys 0..pos inclusive
    o, p = oracle64.attend(cfg, pool, 0, pages, 9, 0, np.zeros(Dh))
    assert np.allclose(o, V[:10, 0].mean(axis=0), atol=1e-12) and np.allclose(p, 0.1)
    # two keys with scores ln 1 and ln 3 -> weights 1/4 and 3/4; also pins the 1/sqrt(Dh) scale
    K2 = np.zeros((2, 1, Dh)); K2[1, 0, 0] = 1.0
    V2 = np.zeros((2, 1, Dh)); V2[0, 0, 0] = 4.0; V2[1, 0, 1] = 8.0
    q = np.zeros(Dh); q[0] = math.log(3.0) * math.sqrt(Dh)
    cfg, pool, pages = _single_seq_cache(oracle64, 2, 1, Dh, K2, V2)
    o, p = oracle64.attend(cfg, pool, 0, pages, 1, 0, q)
    assert np.allclose(p, [0.25, 0.75], atol=1e-12) and np.allclose(o[:2], [1.0, 6.0], atol=1e-12)


def _brute_force_attention(q, K, V, G):
    """Independent 3-loop causal GQA attention in double; q [n, Hq, Dh], K/V [n, Hkv, Dh]."""
    n, Hq, Dh = q.shape
    out = np.zeros_like(q)
    for p in range(n):
        for hq in range(Hq):
            hk = hq // G
            w = np.zeros(n)
            for j in range(n):
                if j <= p:
                    w[j] = math.exp(sum(q[p, hq, e] * K[j, hk, e] for e in range(Dh)) / math.sqrt(Dh))
            w /= w.sum()
            for j in range(n):
                out[p, hq] += w[j] * V[j, hk]
    return out


@pytest.mark.parametrize("page_size", [4, 16])
def test_causal_gqa_brute_force(oracle64, page_size):
    r = np.random.default_rng(7)
    n, Hq, Hkv, Dh = 8, 4, 2, 8
    q = r.standard_normal((n, Hq, Dh))
    K = _bf16_exact(r.standard_normal((n, Hkv, Dh))); V = _bf16_exact(r.standard_normal((n, Hkv, Dh)))
    want = _brute_force_attention(q, K, V, Hq // Hkv)
    perm = [3, 0, 2, 1]
    cfg, pool, pages = _single_seq_cache(oracle64, n, Hkv, Dh, K, V, page_size, perm)
    cfg.n_q_heads = Hq
    for p in range(n):
        for hq in range(Hq):
            o, probs = oracle64.attend(cfg, pool, 0, pages, p, hq, q[p, hq])
            assert probs.shape == (p + 1,)
            assert np.allclose(o, want[p, hq], atol=1e-12), (p, hq)


# ------------------------------------------------------------ whole layer --
SMALL = wl.StageDims(2, 64, 4, 2, 16, 96)


def _torch_reference_single_sequence(dims, weights, x, n_layers, causal=True):
    """float64 composition of library routines for one non-paged sequence starting at position 0."""
    xt = torch.from_numpy(x).double()
    n = xt.shape[0]
    Hq, Hkv, Dh = dims.n_q_heads, dims.n_kv_heads, dims.head_dim
    half = Dh // 2
    ang = torch.arange(n, dtype=torch.float64)[:, None] * torch.pow(
        torch.tensor(dims.rope_base, dtype=torch.float64), -torch.arange(half, dtype=torch.float64) * 2 / Dh)[None]
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]           # [n, 1, half]

    def rope(z):                                                        # z [n, H, Dh]
        zc = torch.complex(z[..., :half], z[..., half:]) * rot
        return torch.cat([zc.real, zc.imag], dim=-1)

    for l in range(n_layers):
        w = {k: torch.from_numpy(v).double() for k, v in weights[l].items()}
        mod = w.get("mod")                                   # [1, 6, d]: one sequence
        sh_a, sc_a, g_a, sh_m, sc_m, g_m = (mod[0, i] for i in range(6)) if mod is not None else (0, 0, 1, 0, 0, 1)
        h = F.rms_norm(xt, (dims.d_model,), w["g_attn"], dims.rms_eps) * (1 + sc_a) + sh_a
        q = rope(F.linear(h, w["w_q"], w.get("b_q")).view(n, Hq, Dh))
        k = rope(F.linear(h, w["w_k"], w.get("b_k")).view(n, Hkv, Dh)).bfloat16().double()
        v = F.linear(h, w["w_v"], w.get("b_v")).view(n, Hkv, Dh).bfloat16().double()
        k = k.repeat_interleave(Hq // Hkv, dim=1); v = v.repeat_interleave(Hq // Hkv, dim=1)
        o = F.scaled_dot_product_attention(q.transpose(0, 1), k.transpose(0, 1), v.transpose(0, 1), is_causal=causal)
        xt = xt + g_a * (o.transpose(0, 1).reshape(n, Hq * Dh) @ w["w_o"].T)
        h2 = F.rms_norm(xt, (dims.d_model,), w["g_mlp"], dims.rms_eps) * (1 + sc_m) + sh_m
        xt = xt + g_m * ((F.silu(h2 @ w["w_gate"].T) * (h2 @ w["w_up"].T)) @ w["w_down"].T)
    return xt.numpy()


@pytest.mark.parametrize("dims,n", [(SMALL, 37), (TINY, 48)])
def test_step_matches_float64_library_composition(oracle32, oracle64, dims, n):
    case = make_case(dims, wl.BatchSpec([n], [0]), seed=3)
    # larger weights than N(0, 0.02) so that attention and the MLP move the output visibly
    weights = [{k: (v if k.startswith("g_") else v * 8.0) for k, v in lw.items()} for lw in case.weights]
    want = _torch_reference_single_sequence(dims, weights, case.x, dims.n_layers)
    assert rel_err(want, case.x) > 0.3          # the layers do something
    y64 = oracle64.step(case.cfg, weights, case.kv_pool.copy(), case.batch.q_len, case.batch.ctx_len,
                        case.block_tables, case.x)
    y32 = oracle32.step(case.cfg, weights, case.kv_pool.copy(), case.batch.q_len, case.batch.ctx_len,
                        case.block_tables, case.x)
    # k and v cross the same bf16 rounding on both sides; float64 agreement is at rounding level
    # (observed 1e-14), float32 at accumulated float32 rounding (observed 4e-6)
    assert rel_err(y64, want) < 1e-10
    assert rel_err(y32, y64) < 5e-5
    # without the cache rounding in play (first layer only, compare a quantity before any
    # read-back): W_o = W_down = 0 gives y = x exactly
    zeroed = [dict(lw, w_o=np.zeros_like(lw["w_o"]), w_down=np.zeros_like(lw["w_down"])) for lw in weights]
    y = oracle32.step(case.cfg, zeroed, case.kv_pool.copy(), case.batch.q_len, case.batch.ctx_len,
                      case.block_tables, case.x)
    assert np.array_equal(y, case.x)


def test_layer_matches_library_when_cache_rounding_is_exact(oracle64):
    """With W_k, W_v chosen so that k and v are exactly representable in bf16 the cache rounding is
    the identity and the agreement with the float64 library composition is at rounding level."""
    dims = wl.StageDims(1, 64, 4, 2, 16, 96)
    case = make_case(dims, wl.BatchSpec([29], [0]), seed=5)
    w = dict(case.weights[0])
    w["w_k"] = np.zeros_like(w["w_k"]); w["w_v"] = np.zeros_like(w["w_v"])   # k = v = 0: exact
    for k in ("w_q", "w_o", "w_gate", "w_up", "w_down"):
        w[k] = w[k] * 8.0
    want = _torch_reference_single_sequence(dims, [w], case.x, 1)
    y = oracle64.step(case.cfg, [w], case.kv_pool.copy(), case.batch.q_len, case.batch.ctx_len,
                      case.block_tables, case.x)
    assert rel_err(y, want) < 1e-12
    assert rel_err(want, case.x) > 0.05


def test_qkv_bias_matches_library_composition_and_closed_form(oracle64):
    """The optional biases of the q, k, v projections enter before RoPE: against torch's linear-with-bias in the
    float64 composition, and, with all three weight matrices zero, against the closed form: every value row is
    b_v, so each head's output is its KV head's slice of b_v whatever the scores are."""
    dims = wl.StageDims(1, 64, 4, 2, 16, 96)
    case = make_case(dims, wl.BatchSpec([23], [0]), seed=8)
    g = np.random.default_rng(8)
    w = {k: (v if k.startswith("g_") else v * 8.0) for k, v in case.weights[0].items()}
    w["b_q"] = g.normal(0, 1.0, dims.n_q_heads * dims.head_dim)
    w["b_k"] = g.normal(0, 1.0, dims.n_kv_heads * dims.head_dim)
    w["b_v"] = g.normal(0, 1.0, dims.n_kv_heads * dims.head_dim)
    args = (case.batch.q_len, case.batch.ctx_len, case.block_tables, case.x)
    y = oracle64.step(case.cfg, [w], case.kv_pool.copy(), *args)
    want = _torch_reference_single_sequence(dims, [w], case.x, 1)
    assert rel_err(y, want) < 1e-10
    no_bias = oracle64.step(case.cfg, [{k: v for k, v in w.items() if not k.startswith("b_")}], case.kv_pool.copy(), *args)
    assert rel_err(y, no_bias) > 0.05           # the biases matter in this case
    for drop in ("b_q", "b_k", "b_v"):          # and each one on its own
        y_drop = oracle64.step(case.cfg, [{k: v for k, v in w.items() if k != drop}], case.kv_pool.copy(), *args)
        assert rel_err(y, y_drop) > 1e-3, drop

    z = dict(w, w_q=np.zeros_like(w["w_q"]), w_k=np.zeros_like(w["w_k"]), w_v=np.zeros_like(w["w_v"]),
             w_down=np.zeros_like(w["w_down"]))
    z["b_v"] = np.asarray(torch.from_numpy(w["b_v"]).bfloat16().double())        # exact in the cache
    y = oracle64.step(case.cfg, [z], case.kv_pool.copy(), *args)
    G = dims.n_q_heads // dims.n_kv_heads
    o_row = np.concatenate([z["b_v"][(hq // G) * dims.head_dim:(hq // G + 1) * dims.head_dim]
                            for hq in range(dims.n_q_heads)])
    want = case.x.astype(np.float64) + (z["w_o"].astype(np.float64) @ o_row)[None, :]
    assert rel_err(y, want) < 1e-12


def test_bidirectional_attention_matches_library_and_invariants(oracle64):
    """The unmasked attention of a denoising-style block: against torch's attention without a causal mask in the
    float64 composition; it differs from the causal result on every row but the last (which sees all keys either
    way); and the mean-pooling closed form: with W_q = 0 every score is 0, so every row's attention output is
    the plain mean of all value rows of the sequence."""
    import dataclasses
    dims = wl.StageDims(2, 64, 4, 2, 16, 96)
    case = make_case(dims, wl.BatchSpec([29], [0]), seed=9)
    weights = [{k: (v if k.startswith("g_") else v * 8.0) for k, v in lw.items()} for lw in case.weights]
    cfg = dataclasses.replace(case.cfg, bidirectional=True)
    args = (case.batch.q_len, case.batch.ctx_len, case.block_tables, case.x)
    y = oracle64.step(cfg, weights, case.kv_pool.copy(), *args)
    want = _torch_reference_single_sequence(dims, weights, case.x, dims.n_layers, causal=False)
    assert rel_err(y, want) < 1e-10
    y_causal = oracle64.step(case.cfg, weights, case.kv_pool.copy(), *args)
    one = dataclasses.replace(cfg, n_layers=1)
    pool1 = case.kv_pool[: one.kv_pool_elems()]
    y1 = oracle64.step(one, weights[:1], pool1.copy(), *args)
    y1c = oracle64.step(dataclasses.replace(one, bidirectional=False), weights[:1], pool1.copy(), *args)
    row_diff = np.max(np.abs(y1 - y1c), axis=1)
    assert row_diff[-1] == 0.0 and np.all(row_diff[:-1] > 1e-6)      # one layer: only the last row sees the same keys
    assert rel_err(y, y_causal) > 0.05

    z = dict(weights[0], w_q=np.zeros_like(weights[0]["w_q"]), w_down=np.zeros_like(weights[0]["w_down"]))
    y0 = oracle64.step(one, [z], pool1.copy(), *args)
    xt = torch.from_numpy(case.x).double()
    h = F.rms_norm(xt, (dims.d_model,), torch.from_numpy(z["g_attn"]).double(), dims.rms_eps)
    v = (h @ torch.from_numpy(z["w_v"]).double().T).bfloat16().double()          # [n, Hkv * Dh], as cached
    G = dims.n_q_heads // dims.n_kv_heads
    o_row = v.mean(dim=0).view(dims.n_kv_heads, dims.head_dim).repeat_interleave(G, dim=0).reshape(-1)
    want0 = xt + (torch.from_numpy(z["w_o"]).double() @ o_row)[None, :]
    assert rel_err(y0, want0.numpy()) < 1e-12


def test_modulation_matches_library_composition_and_special_cases(oracle64):
    """Per-sequence shift / scale / gate vectors of a conditioned block (adaLN-Zero with RMSNorm): against the
    float64 library composition; scale = shift = 0 with gate = 1 is the plain layer, bit for bit; gate = 0 on both
    branches returns the input; and two sequences of one batch each follow their own vectors."""
    dims = wl.StageDims(2, 64, 4, 2, 16, 96)
    case = make_case(dims, wl.BatchSpec([26], [0]), seed=10)
    g = np.random.default_rng(10)
    weights = [{k: (v if k.startswith("g_") else v * 8.0) for k, v in lw.items()} for lw in case.weights]
    mods = [g.normal(0, 0.5, (1, 6, dims.d_model)) for _ in range(dims.n_layers)]
    wm = [dict(lw, mod=m) for lw, m in zip(weights, mods)]
    args = (case.batch.q_len, case.batch.ctx_len, case.block_tables, case.x)
    y = oracle64.step(case.cfg, wm, case.kv_pool.copy(), *args)
    want = _torch_reference_single_sequence(dims, wm, case.x, dims.n_layers)
    assert rel_err(y, want) < 1e-10
    y_plain = oracle64.step(case.cfg, weights, case.kv_pool.copy(), *args)
    assert rel_err(y, y_plain) > 0.05
    ident = np.zeros((1, 6, dims.d_model)); ident[0, 2] = 1.0; ident[0, 5] = 1.0
    assert np.array_equal(oracle64.step(case.cfg, [dict(lw, mod=ident) for lw in weights], case.kv_pool.copy(), *args),
                          y_plain)
    closed = np.array(mods[0]); closed[0, 2] = 0.0; closed[0, 5] = 0.0
    y0 = oracle64.step(case.cfg, [dict(lw, mod=closed) for lw in weights], case.kv_pool.copy(), *args)
    assert np.array_equal(y0, case.x.astype(y0.dtype))
    for drop in range(6):                        # every one of the six vectors matters on its own
        m2 = [np.array(m) for m in mods]
        m2[0][0, drop] = 1.0 if drop in (2, 5) else 0.0
        y2 = oracle64.step(case.cfg, [dict(lw, mod=m) for lw, m in zip(weights, m2)], case.kv_pool.copy(), *args)
        assert rel_err(y2, y) > 1e-3, drop

    # two sequences in one batch: each equals the single-sequence run with its own vectors
    one = wl.StageDims(1, 64, 4, 2, 16, 96)
    both = make_case(one, wl.BatchSpec([13, 21], [0, 0]), seed=12)
    m_both = g.normal(0, 0.5, (2, 6, one.d_model))
    w1 = {k: (v if k.startswith("g_") else v * 8.0) for k, v in both.weights[0].items()}
    y_both = oracle64.step(both.cfg, [dict(w1, mod=m_both)], both.kv_pool.copy(), both.batch.q_len, both.batch.ctx_len,
                           both.block_tables, both.x)
    t0 = 0
    for s_i, n in enumerate([13, 21]):
        want_s = _torch_reference_single_sequence(one, [dict(w1, mod=m_both[s_i:s_i + 1])], both.x[t0:t0 + n], 1)
        assert rel_err(y_both[t0:t0 + n], want_s) < 1e-10
        t0 += n


def test_zero_gate_weight_means_mlp_adds_nothing(oracle32):
    case = make_case(SMALL, wl.BatchSpec([11], [0]), seed=6)
    w0 = [dict(lw, w_gate=np.zeros_like(lw["w_gate"])) for lw in case.weights]
    w1 = [dict(lw, w_gate=np.zeros_like(lw["w_gate"]), w_down=np.zeros_like(lw["w_down"])) for lw in case.weights]
    args = (case.batch.q_len, case.batch.ctx_len, case.block_tables, case.x)
    assert np.array_equal(oracle32.step(case.cfg, w0, case.kv_pool.copy(), *args),
                          oracle32.step(case.cfg, w1, case.kv_pool.copy(), *args))


def test_future_tokens_do_not_change_earlier_rows(oracle32):
    case = make_case(SMALL, wl.BatchSpec([20], [0]), seed=7)
    args = (case.batch.q_len, case.batch.ctx_len, case.block_tables)
    y0 = oracle32.step(case.cfg, case.weights, case.kv_pool.copy(), *args, case.x)
    x2 = case.x.copy(); x2[13:] += 1.0
    y1 = oracle32.step(case.cfg, case.weights, case.kv_pool.copy(), *args, x2)
    assert np.array_equal(y0[:13], y1[:13])
    assert not np.array_equal(y0[13], y1[13])


def test_gqa_equals_mha_with_duplicated_kv_heads(oracle32):
    dims = SMALL
    case = make_case(dims, wl.BatchSpec([17, 1], [0, 9]), seed=8, kv_fill=True)
    G = dims.n_q_heads // dims.n_kv_heads
    mha = wl.StageDims(dims.n_layers, dims.d_model, dims.n_q_heads, dims.n_q_heads, dims.head_dim, dims.d_ffn)
    dup = lambda w: np.repeat(w.reshape(dims.n_kv_heads, dims.head_dim, -1), G, axis=0).reshape(-1, w.shape[1])
    w_mha = [dict(lw, w_k=dup(lw["w_k"]), w_v=dup(lw["w_v"])) for lw in case.weights]
    pool = case.kv_pool.reshape(dims.n_layers, 2, case.cfg.num_pages, dims.n_kv_heads, dims.page_size, dims.head_dim)
    pool_mha = np.repeat(pool, G, axis=3).reshape(-1).copy()
    args = (case.batch.q_len, case.batch.ctx_len, case.block_tables, case.x)
    y_gqa = oracle32.step(case.cfg, case.weights, case.kv_pool.copy(), *args)
    y_mha = oracle32.step(oracle_cfg(mha, case.cfg.num_pages), w_mha, pool_mha, *args)
    assert np.array_equal(y_gqa, y_mha)


# --------------------------------------------------------------- paging --
def test_physical_page_permutation_and_page_size_leave_y_unchanged(oracle32):
    dims = SMALL
    batch = wl.BatchSpec([21, 33, 1], [0, 16, 40])
    base = make_case(dims, batch, seed=9)
    # context of sequences 1 and 2 is written by an earlier oracle step
    pre = wl.BatchSpec([16, 40], [0, 0])
    x_pre = wl.to_f32_numpy(wl.make_x(pre.n_tokens, dims.d_model, 9, index=1))

    def run(page_size, perm_seed):
        d = wl.StageDims(dims.n_layers, dims.d_model, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.d_ffn,
                         page_size=page_size)
        num_pages = wl.pages_needed(batch, page_size) + 5
        alloc = PageAllocator(num_pages, page_size)
        tables = [alloc.alloc(s, t) for s, t in enumerate(batch.total_len())]
        if perm_seed is not None:
            perm = np.random.default_rng(perm_seed).permutation(num_pages)
            tables = [[int(perm[p]) for p in t] for t in tables]
        bt = block_table_array(tables, max(len(t) for t in tables) + 1)
        cfg = oracle_cfg(d, num_pages)
        pool = np.full(cfg.kv_pool_elems(), 0x7fc0, dtype=np.uint16)
        oracle32.step(cfg, base.weights, pool, pre.q_len, pre.ctx_len, bt[1:], x_pre)
        y = oracle32.step(cfg, base.weights, pool, batch.q_len, batch.ctx_len, bt, base.x)
        # pages that no sequence owns keep their canary
        owned = sorted(p for t in tables for p in t)
        pool6 = pool.reshape(d.n_layers, 2, num_pages, d.n_kv_heads, page_size, d.head_dim)
        for p in range(num_pages):
            if p not in owned:
                assert np.all(pool6[:, :, p] == 0x7fc0)
        return y

    y_ref = run(16, None)
    assert np.all(np.isfinite(y_ref))
    for page_size, perm_seed in ((16, 1), (16, 2), (8, None), (32, 3), (4, 4)):
        assert np.array_equal(run(page_size, perm_seed), y_ref), (page_size, perm_seed)


# -------------------------------------------------------------- chunking --
def _run_chunks(orc, case_full, chunks):
    """Feeds one sequence's tokens in the given chunk sizes; returns all output rows."""
    pool = case_full.kv_pool.copy()
    rows, done = [], 0
    for n in chunks:
        y = orc.step(case_full.cfg, case_full.weights, pool, [n], [done], case_full.block_tables,
                     case_full.x[done:done + n])
        rows.append(y)
        done += n
    return np.concatenate(rows), pool


@pytest.mark.parametrize("chunks", [(16, 32), (1, 47), (47, 1), (7, 9, 32), tuple([1] * 48)])
def test_chunked_prefill_equals_full_prefill(oracle32, chunks):
    case = make_case(TINY, wl.BatchSpec([48], [0]), seed=0)
    y_full, pool_full = _run_chunks(oracle32, case, (48,))
    y_chunk, pool_chunk = _run_chunks(oracle32, case, chunks)
    # in-chunk keys are read back from the bf16 cache in both runs -> bit-identical
    assert np.array_equal(y_full, y_chunk)
    assert np.array_equal(pool_full, pool_chunk)


def test_decode_step_equals_last_row_of_prefill(oracle32):
    case = make_case(TINY, wl.BatchSpec([41], [0]), seed=1)
    y_full, _ = _run_chunks(oracle32, case, (41,))
    y_two, _ = _run_chunks(oracle32, case, (40, 1))
    assert np.array_equal(y_two[40], y_full[40])


def test_batch_composition_independence(oracle32):
    dims = TINY
    batch = wl.make_batch("c1_tiny", 0)
    case = make_case(dims, batch, seed=0, kv_fill=True)
    y_mixed = oracle32.step(case.cfg, case.weights, case.kv_pool.copy(), batch.q_len, batch.ctx_len,
                            case.block_tables, case.x)
    t0 = 0
    for s in range(batch.n_seqs):
        n = batch.q_len[s]
        y_alone = oracle32.step(case.cfg, case.weights, case.kv_pool.copy(), [n], [batch.ctx_len[s]],
                                case.block_tables[s:s + 1], case.x[t0:t0 + n])
        assert np.array_equal(y_alone, y_mixed[t0:t0 + n]), s
        t0 += n


def test_row_mask_matches_full_evaluation(oracle32):
    batch = wl.make_batch("c1_tiny", 0)
    case = make_case(TINY, batch, seed=0, kv_fill=True)
    args = (batch.q_len, batch.ctx_len, case.block_tables, case.x)
    pool_a, pool_b = case.kv_pool.copy(), case.kv_pool.copy()
    y_full = oracle32.step(case.cfg, case.weights, pool_a, *args)
    mask = np.zeros(batch.n_tokens, dtype=np.uint8); mask[[0, 31, 32, 79, 80, 81]] = 1
    y_mask = oracle32.step(case.cfg, case.weights, pool_b, *args, last_layer_row_mask=mask)
    sel = mask.astype(bool)
    assert np.array_equal(y_mask[sel], y_full[sel])
    assert np.array_equal(pool_a, pool_b)


def test_kv_pre_is_k_after_rope_and_v_before_the_cache_rounding(oracle32, oracle64):
    """kv_pre, the layer's side output that the GPU tests hold the written K / V against: slot 0 must be
    rope(h W_k^T + b_k) and slot 1 h W_v^T + b_v, formed here from the separately pinned primitives (rmsnorm,
    linear, rope), and its bf16 rounding must be the very bits the same call wrote into the cache -- a copy taken
    before RoPE, K and V swapped, or a wrong page / slot fails one of the two."""
    batch = wl.make_batch("c1_tiny", 0)                    # prefill 32, 48 + decode with ctx 40, 64
    for orc, tol in ((oracle32, 0.0), (oracle64, 0.0)):
        case = make_case(TINY, batch, seed=0, kv_fill=True)
        w = dict(case.weights[0])
        g = np.random.default_rng(4)
        w["b_k"] = g.normal(0, 0.5, TINY.kv_dim).astype(np.float32)
        w["b_v"] = g.normal(0, 0.5, TINY.kv_dim).astype(np.float32)
        pool = case.kv_pool.copy()
        _, kv_pre = orc.layer(case.cfg, w, 0, pool, batch.q_len, batch.ctx_len, case.block_tables, case.x,
                              want_kv_pre=True)
        assert kv_pre.shape == (batch.n_tokens, 2, TINY.kv_dim)
        h = orc.rmsnorm(case.x, w["g_attn"], TINY.rms_eps)
        k_lin = orc.linear(h, w["w_k"]) + w["b_k"].astype(orc.dtype)
        v_lin = orc.linear(h, w["w_v"]) + w["b_v"].astype(orc.dtype)
        pool5 = pool.reshape(TINY.n_layers, 2, case.cfg.num_pages, TINY.n_kv_heads, 16, TINY.head_dim)
        t = 0
        moved = 0.0
        for s in range(batch.n_seqs):
            for j in range(batch.q_len[s]):
                pos = batch.ctx_len[s] + j
                k_rot = orc.rope(k_lin[t].reshape(TINY.n_kv_heads, TINY.head_dim), pos, TINY.rope_base)
                assert np.array_equal(kv_pre[t, 0], k_rot.reshape(-1)), (s, j)
                assert np.array_equal(kv_pre[t, 1], v_lin[t]), (s, j)
                moved = max(moved, float(np.max(np.abs(k_rot.reshape(-1) - k_lin[t]))))
                page, slot = case.block_tables[s, pos // 16], pos % 16
                for kv in (0, 1):
                    want = np.array([orc.bf16_rne(float(v)) for v in kv_pre[t, kv]], dtype=np.uint16)
                    assert np.array_equal(pool5[0, kv, page, :, slot, :].reshape(-1), want), (s, j, kv)
                t += 1
        assert moved > 0.1                                  # the rotation is visible: "before RoPE" would fail
        assert float(np.max(np.abs(kv_pre[:, 0] - kv_pre[:, 1]))) > 0.1   # and K is not V


# --------------------------------------------------- float32 vs float64 --
def test_float32_oracle_is_close_to_float64_on_config_1(oracle32, oracle64):
    batch = wl.make_batch("c1_tiny", 0)
    case = make_case(TINY, batch, seed=0, kv_fill=True)
    args = (batch.q_len, batch.ctx_len, case.block_tables, case.x)
    y32 = oracle32.step(case.cfg, case.weights, case.kv_pool.copy(), *args)
    y64 = oracle64.step(case.cfg, case.weights, case.kv_pool.copy(), *args)
    assert rel_err(y32, y64) < 1e-3      # dominated by 1-ulp flips of cached bf16 values
    assert rel_err(y64, case.x) > 1e-2   # and the layer is not the identity


def test_operand_rounding_diagnostic_is_off_by_default_and_fp16_is_the_finer_grid(oracle32):
    """The diagnostic switch (never the pass/fail oracle): off by default, rounding the intermediates moves
    the output, and the fp16 grid for h, o and act (11-bit significand) moves it less than bf16 (8-bit)."""
    from oracle.oracle import ROUND_ALL, ROUND_ACT_F16
    dims = wl.StageDims(2, 128, 4, 2, 32, 512)
    case = make_case(dims, wl.BatchSpec([24, 9], [0, 0]), seed=21)
    args = (case.cfg, case.weights, None, case.batch.q_len, case.batch.ctx_len, case.block_tables, case.x)

    def run(mask):
        oracle32.set_operand_rounding(mask)
        try:
            return oracle32.step(args[0], args[1], case.kv_pool.copy(), *args[3:])
        finally:
            oracle32.set_operand_rounding(0)

    y0, y0_again = run(0), run(0)
    assert np.array_equal(y0, y0_again)
    e_bf16, e_f16 = rel_err(run(ROUND_ALL), y0), rel_err(run(ROUND_ALL | ROUND_ACT_F16), y0)
    assert 0 < e_f16 < e_bf16 < 2e-2
    # h, o, act alone: the two grids differ by 2^3 in spacing (1-ulp flips of cached bf16 K/V blur the ratio)
    e_b, e_h = rel_err(run(1 | 8 | 16), y0), rel_err(run(1 | 8 | 16 | ROUND_ACT_F16), y0)
    assert e_b / 16 < e_h < e_b / 2
