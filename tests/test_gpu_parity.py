"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.

Tolerances (from the arithmetic: bf16 tensor-core operands, fp32 accumulation, fp32 residual stream):
  y_out      max |y_gpu - y_oracle| <= 2e-2 * RMS(y_oracle), per tensor;
  K/V bytes  each element written this step against the oracle's value BEFORE its bf16 rounding:
             |k_gpu - k_ref| <= 2^-8 |k_ref| + 1e-2 RMS(k_ref) (one bf16 rounding plus operand noise; two
             independently rounded bf16 tensors legitimately differ by an ulp in many elements);
  integers   block tables, slots, and the set of cache bytes a step touches: bit-exact;
  budgets    y_out and the whole KV pool bit-identical for every sm_budget.
"""
import numpy as np
import pytest
import torch

from oracle.oracle import Oracle
from paper_2608_01785_b200 import binding as B
from paper_2608_01785_b200 import workloads as wl
from tests.gpu_helpers import bits_to_f32, make_stage, run_step
from tests.helpers import make_case, rel_err

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.fixture(scope="module")
def orc():
    return Oracle("f32")


def one_layer(dims):
    return wl.StageDims(1, dims.d_model, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.d_ffn)


def check_kv_written(case, pool_in, pool_gpu, kv_pre, layer=0):
    """Slots of `layer` written by the step obey the element rule; every other byte of the pool is unchanged."""
    d = case.dims
    shape = (d.n_layers, 2, case.cfg.num_pages, d.n_kv_heads, d.page_size, d.head_dim)
    g = bits_to_f32(pool_gpu).reshape(shape)
    touched = np.zeros(shape, dtype=bool)
    t = 0
    for s, (n, c) in enumerate(zip(case.batch.q_len, case.batch.ctx_len)):
        for j in range(n):
            p = c + j
            page, slot = case.block_tables[s, p // 16], p % 16
            touched[:, :, page, :, slot, :] = True
            for kv in range(2):
                ref = kv_pre[t, kv].reshape(d.n_kv_heads, d.head_dim).astype(np.float64)
                got = g[layer, kv, page, :, slot, :].astype(np.float64)
                rms = np.sqrt(np.mean(kv_pre[:, kv].astype(np.float64) ** 2))
                bound = 2.0 ** -8 * np.abs(ref) + 1e-2 * rms
                assert np.all(np.abs(got - ref) <= bound), (s, j, kv, float(np.max(np.abs(got - ref) / bound)))
            t += 1
    untouched = ~touched.reshape(-1)
    assert np.array_equal(pool_gpu[untouched], pool_in[untouched]), "bytes outside the step's slots changed"


# ----------------------------------------------------------------- GEMM op --
@pytest.mark.parametrize("M,N,K,resid", [(128, 256, 64, False), (82, 520, 200, True), (300, 264, 72, True),
                                         (2112, 1024, 3584, False), (1000, 2048, 1408, True), (16, 1536, 1024, True),
                                         # at most 64 rows and few output tiles: the weight-streaming kernel,
                                         # with one, two and four 16-row tiles and a ragged last tile
                                         (1, 256, 1024, True), (33, 512, 2048, True), (48, 1024, 4096, False),
                                         (64, 3584, 3584, True),
                                         # tile counts that leave the last round of the 74 pairs ragged: the K blocks
                                         # are cut into equal runs (stream-K form), partial sums added in K order
                                         (2112, 3584, 4096, True), (2900, 2048, 4608, False), (1500, 3328, 4224, True)])
@pytest.mark.parametrize("a_dtype", [torch.bfloat16, torch.float16])
def test_gemm_op_matches_oracle_and_is_budget_invariant(orc, M, N, K, resid, a_dtype):
    """Both operand forms: bf16 x bf16, and the fp16 x fp16 form the stage uses by default."""
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(M * 7 + N)
    a = torch.randn(M, K, generator=g).to(a_dtype)
    w = (torch.randn(N, K, generator=g) * 0.02).to(a_dtype)
    r = torch.randn(M, N, generator=g) if resid else None
    want = orc.linear(a.float().numpy(), w.float().numpy())
    if resid:
        want = want + r.numpy()
    outs = []
    a_d, w_d = a.to(dev), w.to(dev)
    stream_k = M * N >= 1500 * 3328
    for budget in (148, 74, 37, 8, 1):
        if budget == 1 and M * N > 300 * 600 and not (stream_k and a_dtype == torch.float16):
            continue
        out = torch.full((M, N), float("nan"), device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        r_d = r.to(dev) if resid else None
        B.hs_op_gemm_bf16(a_d.data_ptr(), w_d.data_ptr(), r_d.data_ptr() if resid else 0, out.data_ptr(), M, N, K,
                          budget, status.data_ptr(), a_is_f16=a_dtype == torch.float16)
        torch.cuda.synchronize()
        assert status.item() == 0
        outs.append(out.cpu())
    assert rel_err(outs[0].numpy(), want) < 1e-4          # fp32 accumulation of exact 16-bit products
    for o in outs[1:]:
        assert torch.equal(o, outs[0])


def test_gemm_op_in_place_residual(orc):
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(5)
    a = torch.randn(200, 320, generator=g).to(torch.bfloat16)
    w = torch.randn(264, 320, generator=g).to(torch.bfloat16)
    x = torch.randn(200, 264, generator=g)
    want = x.numpy() + orc.linear(a.float().numpy(), w.float().numpy())
    x_d, a_d, w_d = x.to(dev), a.to(dev), w.to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.hs_op_gemm_bf16(a_d.data_ptr(), w_d.data_ptr(), x_d.data_ptr(), x_d.data_ptr(), 200, 264, 320, 148,
                      status.data_ptr())
    torch.cuda.synchronize()
    assert rel_err(x_d.cpu().numpy(), want) < 1e-4


def test_gemm_op_argument_errors():
    dev = torch.device("cuda:0")
    buf = torch.zeros(1 << 16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    p = buf.data_ptr()
    for args, code in (((p, p, 0, p, 16, 20, 64, 148), B.HS_ERR_UNSUPPORTED_SHAPE),      # N % 8
                       ((p, p, 0, p, 16, 64, 60, 148), B.HS_ERR_UNSUPPORTED_SHAPE),      # K % 8
                       ((p, p, 0, p, 16, 64, 64, 0), B.HS_ERR_INVALID_BUDGET),
                       ((p, p, 0, p, 16, 64, 64, 149), B.HS_ERR_INVALID_BUDGET),
                       ((0, p, 0, p, 16, 64, 64, 148), B.HS_ERR_INVALID_ARG)):
        with pytest.raises(B.HsError) as e:
            B.hs_op_gemm_bf16(*args, status.data_ptr())
        assert e.value.status == code


# ---------------------------------------------------------------- config 1 --
def config1_case(orc):
    """Config 1 with a self-consistent cache: the decode sequences' context (40 and 64 tokens) is written
    by an oracle prefill step, and that pool is what both sides start the step under test from."""
    dims = wl.DIMS["c1_tiny"]
    batch = wl.make_batch("c1_tiny", 0)
    case = make_case(dims, batch, seed=0)
    pre = wl.BatchSpec([40, 64], [0, 0])
    x_pre = wl.to_f32_numpy(wl.make_x(pre.n_tokens, dims.d_model, 0, index=1))
    orc.step(case.cfg, case.weights, case.kv_pool, pre.q_len, pre.ctx_len, case.block_tables[2:], x_pre)
    return case


@pytest.mark.parametrize("flags", [0, B.HS_FLAG_BF16_ACTIVATIONS])
def test_config1_step_matches_oracle_at_budgets_148_and_8(orc, flags):
    """flags 0: h, o and act in fp16 against fp16 copies of the weights (the default); the flag: all bf16."""
    case = config1_case(orc)
    assert case.block_tables[:, :5].tolist() == [[0, 1, -1, -1, -1], [2, 3, 4, -1, -1], [5, 6, 7, -1, -1],
                                                 [8, 9, 10, 11, 12]]
    pool_ref = case.kv_pool.copy()
    y_ref, kv_pre = orc.layer(case.cfg, case.weights[0], 0, pool_ref, case.batch.q_len, case.batch.ctx_len,
                              case.block_tables, case.x, want_kv_pre=True)
    results = []
    for budget in (148, 8):
        st = make_stage(case, flags=flags)
        y, pool = run_step(st, case, budget)
        st.close()
        err = rel_err(y, y_ref)
        print(f"config 1 (flags {flags}), sm_budget {budget}: max|err|/RMS = {err:.2e}")
        assert err <= TOL
        check_kv_written(case, case.kv_pool, pool, kv_pre)
        results.append((y, pool))
    assert np.array_equal(results[0][0], results[1][0]) and np.array_equal(results[0][1], results[1][1])


def test_budget_errors_and_idempotence(orc):
    case = config1_case(orc)
    st = make_stage(case)
    try:
        y1, pool1 = run_step(st, case, 148)
        y2, pool2 = run_step(st, case, 3)            # same step again: same slots, same values
        assert np.array_equal(y1, y2) and np.array_equal(pool1, pool2)
        x = case.x_t.to(st.device)
        y = torch.empty(case.batch.n_tokens, case.dims.d_model, device=st.device)
        b = st.make_batch(case.batch.q_len, case.batch.ctx_len, case.block_tables, x, y)
        for budget in (0, -1, st.sm_count + 1):
            with pytest.raises(B.HsError) as e:
                st.step(b, budget)
            assert e.value.status == B.HS_ERR_INVALID_BUDGET
        bad = case.block_tables.copy(); bad[0, 0] = case.cfg.num_pages
        with pytest.raises(B.HsError) as e:
            st.step(st.make_batch(case.batch.q_len, case.batch.ctx_len, bad, x, y), 8)
        assert e.value.status == B.HS_ERR_BAD_BLOCK_TABLE
        torch.cuda.synchronize()
        assert np.array_equal(wl.bf16_bits_numpy(st.kv_pool).reshape(-1), pool1)   # nothing was launched
    finally:
        st.close()


# -------------------------------------------------------------- edge cases --
EDGE = {
    # name: (dims, q_len, ctx_len)
    "single_token_prompt": (wl.StageDims(1, 256, 4, 2, 64, 688), [1], [0]),
    "page_boundaries": (wl.StageDims(1, 256, 4, 2, 64, 688), [16, 17, 15, 1, 1, 1], [0, 16, 1, 15, 16, 31]),
    "continuation_chunks": (wl.StageDims(2, 256, 4, 2, 64, 688), [40, 100, 7], [24, 60, 129]),
    "head_dim_128_mha": (wl.StageDims(1, 256, 2, 2, 128, 512), [70, 1, 33], [0, 200, 5]),
    "gqa_7_dh128": (wl.StageDims(1, 512, 7, 1, 128, 1024), [61, 1, 1, 19], [3, 90, 700, 64]),
    "gqa_16_dh64": (wl.StageDims(1, 256, 32, 2, 64, 256), [24, 1], [9, 130]),
    "long_decode_many_splits": (wl.StageDims(1, 256, 4, 2, 64, 688), [1, 1, 1], [511, 512, 2100]),
    "long_prefill_dh128": (wl.StageDims(1, 256, 8, 1, 128, 640), [700, 1], [0, 1500]),
    "many_sequences": (wl.StageDims(1, 256, 4, 2, 64, 688), [1] * 40 + [3] * 10, list(range(0, 400, 10)) + [5] * 10),
    "two_layers_talker_like": (wl.StageDims(2, 1024, 16, 4, 64, 2816), [1] * 16, [128 + 57 * i for i in range(16)]),
    # few tokens against a long K: the QKV and gate/up GEMMs split K four ways through the scratch tile
    "small_step_split_k": (wl.StageDims(1, 2048, 8, 2, 128, 1024), [20, 1, 1], [0, 300, 17]),
    # the RoPE base of long-context checkpoints, positions up to 3000
    "rope_base_1e6": (wl.StageDims(1, 256, 4, 2, 64, 688, rope_base=1.0e6), [90, 1, 1], [0, 2999, 1500]),
    # rows too wide for the bulk-staged RMSNorm (register-staged fallback), K split eight ways
    "wide_rows_d8192": (wl.StageDims(1, 8192, 2, 2, 64, 128), [20, 1], [0, 37]),
}


@pytest.mark.parametrize("name", sorted(EDGE))
def test_edge_cases_match_oracle(orc, name):
    dims, q_len, ctx_len = EDGE[name]
    batch = wl.BatchSpec(list(q_len), list(ctx_len))
    case = make_case(dims, batch, seed=11, kv_fill=True)
    # the tail of every sequence's last page (and every page nobody owns) holds NaN on entry: it must
    # neither reach the output nor be written
    # view [layer][K|V][kv_head][page][slot][Dh] so that a [page, slot] mask indexes it
    pool6 = case.kv_pool.reshape(dims.n_layers, 2, case.cfg.num_pages, dims.n_kv_heads, 16,
                                 dims.head_dim).transpose(0, 1, 3, 2, 4, 5)
    owned = np.zeros((case.cfg.num_pages, 16), dtype=bool)
    for s, c in enumerate(batch.ctx_len):
        for p in range(c):
            owned[case.block_tables[s, p // 16], p % 16] = True
    pool6[:, :, :, ~owned] = 0x7fc0
    pool_ref = case.kv_pool.copy()
    y_ref = orc.step(case.cfg, case.weights, pool_ref, batch.q_len, batch.ctx_len, case.block_tables, case.x)
    assert np.all(np.isfinite(y_ref))
    outs = []
    # more than one 128-row tile per GEMM (two m-tiles, K splits over several tiles); also run on a single SM
    budgets = (148, 5, 1) if name == "continuation_chunks" else (148, 5)
    for budget in budgets:
        st = make_stage(case)
        y, pool = run_step(st, case, budget)
        st.close()
        err = rel_err(y, y_ref)
        print(f"{name}, sm_budget {budget}: max|err|/RMS = {err:.2e}")
        assert err <= TOL
        outs.append((y, pool))
        # canary slots that the step does not own are untouched
        written = np.zeros_like(owned)
        for s, (n, c) in enumerate(zip(batch.q_len, batch.ctx_len)):
            for p in range(c, c + n):
                written[case.block_tables[s, p // 16], p % 16] = True
        g6 = pool.reshape(dims.n_layers, 2, case.cfg.num_pages, dims.n_kv_heads, 16,
                          dims.head_dim).transpose(0, 1, 3, 2, 4, 5)
        assert np.all(g6[:, :, :, ~(owned | written)] == 0x7fc0)
        assert np.array_equal(g6[:, :, :, owned & ~written], pool6[:, :, :, owned & ~written])
    for other in outs[1:]:
        assert np.array_equal(outs[0][0], other[0]) and np.array_equal(outs[0][1], other[1])
    # the all-bf16 variant of the stage (no fp16 weight copies) on the same case
    st = make_stage(case, flags=B.HS_FLAG_BF16_ACTIVATIONS)
    y, _ = run_step(st, case, 148)
    st.close()
    err = rel_err(y, y_ref)
    print(f"{name}, bf16 activations: max|err|/RMS = {err:.2e}")
    assert err <= TOL


BIAS_CASES = {
    # name: (dims, q_len, ctx_len): which QKV epilogue adds the biases
    "two_row_tiles_dh64": (wl.StageDims(2, 256, 4, 2, 64, 688), [100, 60, 1, 1], [0, 37, 64, 200]),   # T > 128
    "single_tile_dh128": (wl.StageDims(1, 256, 2, 2, 128, 512), [70, 1, 33], [0, 200, 5]),          # 64 < T <= 128
    "streaming_kernel_dh64": (wl.StageDims(2, 1024, 16, 4, 64, 2816), [1] * 16, [128 + 57 * i for i in range(16)]),
    "streaming_kernel_dh128": (wl.StageDims(1, 2048, 8, 2, 128, 1024), [20, 1, 1], [0, 300, 17]),
}


@pytest.mark.parametrize("name", sorted(BIAS_CASES))
def test_qkv_bias_matches_oracle(orc, name):
    """Biases on q, k and v (N(0, 0.5): as large as the projections themselves) in every variant of the QKV
    epilogue; the same step with one bias missing follows the oracle with that bias missing, so none of the
    three is dropped or attached to the wrong projection."""
    dims, q_len, ctx_len = BIAS_CASES[name]
    batch = wl.BatchSpec(list(q_len), list(ctx_len))
    case = make_case(dims, batch, seed=21, kv_fill=True)
    g = torch.Generator().manual_seed(77)
    q_dim, kv_dim = dims.n_q_heads * dims.head_dim, dims.n_kv_heads * dims.head_dim
    biases = [[(torch.randn(n, generator=g) * 0.5).to(torch.bfloat16) for n in (q_dim, kv_dim, kv_dim)]
              for _ in range(dims.n_layers)]
    weights = [dict(lw, b_q=b[0].float().numpy(), b_k=b[1].float().numpy(), b_v=b[2].float().numpy())
               for lw, b in zip(case.weights, biases)]
    y_ref = orc.step(case.cfg, weights, case.kv_pool.copy(), batch.q_len, batch.ctx_len, case.block_tables, case.x)
    y_plain = orc.step(case.cfg, case.weights, case.kv_pool.copy(), batch.q_len, batch.ctx_len, case.block_tables,
                       case.x)
    assert rel_err(y_plain, y_ref) > 0.05
    outs = []
    for budget in (148, 5):
        st = make_stage(case)
        dev_b = [[t.to(st.device) for t in b] for b in biases]
        for l, b in enumerate(dev_b):
            st.set_qkv_bias(l, *b)
        y, pool = run_step(st, case, budget)
        err = rel_err(y, y_ref)
        print(f"{name}, sm_budget {budget}: max|err|/RMS = {err:.2e}")
        assert err <= TOL
        outs.append((y, pool))
        if budget == 148:
            for drop, key in enumerate(("b_q", "b_k", "b_v")):
                w_drop = [{k: v for k, v in weights[0].items() if k != key}] + weights[1:]
                y_ref_drop = orc.step(case.cfg, w_drop, case.kv_pool.copy(), batch.q_len, batch.ctx_len,
                                      case.block_tables, case.x)
                assert rel_err(y_ref_drop, y_ref) > 5e-3, key      # the missing bias is visible in the oracle
                st.kv_pool.copy_(wl.bits_to_bf16_tensor(case.kv_pool, st.device))
                st.set_qkv_bias(0, *[None if i == drop else t for i, t in enumerate(dev_b[0])])
                y_drop, _ = run_step(st, case, budget)
                assert rel_err(y_drop, y_ref_drop) <= TOL, key     # and the GPU follows it
        st.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


BIDIR_CASES = {
    # name: (dims, q_len, ctx_len)
    "dh64_several_sequences": (wl.StageDims(2, 256, 4, 2, 64, 688), [100, 37, 1, 64], [0, 0, 0, 0]),
    "dh128_with_cached_context": (wl.StageDims(1, 256, 2, 2, 128, 512), [70, 20, 1], [0, 33, 40]),
    "gqa_8_long": (wl.StageDims(1, 256, 8, 1, 128, 640), [300], [0]),
}


@pytest.mark.parametrize("name", sorted(BIDIR_CASES))
def test_bidirectional_attention_matches_oracle(orc, name):
    """HS_FLAG_BIDIRECTIONAL: no causal mask (the attention of a denoising-style block).  Early rows now depend on
    later tokens of their sequence, so the result must differ from the causal one on those rows."""
    import dataclasses
    dims, q_len, ctx_len = BIDIR_CASES[name]
    batch = wl.BatchSpec(list(q_len), list(ctx_len))
    case = make_case(dims, batch, seed=31, kv_fill=True)
    cfg = dataclasses.replace(case.cfg, bidirectional=True)
    y_ref = orc.step(cfg, case.weights, case.kv_pool.copy(), batch.q_len, batch.ctx_len, case.block_tables, case.x)
    y_causal = orc.step(case.cfg, case.weights, case.kv_pool.copy(), batch.q_len, batch.ctx_len, case.block_tables,
                        case.x)
    assert rel_err(y_causal, y_ref) > 5 * TOL
    outs = []
    for budget in (148, 5):
        st = make_stage(case, flags=B.HS_FLAG_BIDIRECTIONAL)
        y, pool = run_step(st, case, budget)
        st.close()
        err = rel_err(y, y_ref)
        print(f"{name}, sm_budget {budget}: max|err|/RMS = {err:.2e}")
        assert err <= TOL
        outs.append((y, pool))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


MOD_CASES = {
    # name: (dims, q_len, ctx_len, flags)
    "two_row_tiles_bidirectional": (wl.StageDims(2, 256, 4, 4, 64, 688), [150, 60, 9], [0, 0, 0], B.HS_FLAG_BIDIRECTIONAL),
    "single_tile_causal": (wl.StageDims(1, 256, 2, 2, 128, 512), [70, 1, 33], [0, 200, 5], 0),
    "streaming_kernel_16_rows": (wl.StageDims(2, 1024, 16, 4, 64, 2816), [1] * 16, [128 + 57 * i for i in range(16)], 0),
    "streaming_kernel_22_rows": (wl.StageDims(1, 2048, 8, 2, 128, 1024), [20, 1, 1], [0, 300, 17], 0),
    "wide_rows_d8192": (wl.StageDims(1, 8192, 2, 2, 64, 128), [20, 1], [0, 37], 0),
}


@pytest.mark.parametrize("name", sorted(MOD_CASES))
def test_modulation_matches_oracle(orc, name):
    """Per-sequence shift / scale / gate vectors (hs_stage_set_modulation) through both RMSNorm kernels and every
    variant of the residual GEMM epilogue; switching the modulation off again restores the plain step."""
    import dataclasses
    dims, q_len, ctx_len, flags = MOD_CASES[name]
    batch = wl.BatchSpec(list(q_len), list(ctx_len))
    case = make_case(dims, batch, seed=41, kv_fill=True)
    cfg = dataclasses.replace(case.cfg, bidirectional=bool(flags & B.HS_FLAG_BIDIRECTIONAL))
    g = torch.Generator().manual_seed(99)
    mod = torch.randn(dims.n_layers, batch.n_seqs, 6, dims.d_model, generator=g) * 0.5
    weights = [dict(lw, mod=mod[l].numpy()) for l, lw in enumerate(case.weights)]
    y_ref = orc.step(cfg, weights, case.kv_pool.copy(), batch.q_len, batch.ctx_len, case.block_tables, case.x)
    y_plain = orc.step(cfg, case.weights, case.kv_pool.copy(), batch.q_len, batch.ctx_len, case.block_tables, case.x)
    assert rel_err(y_plain, y_ref) > 5 * TOL
    outs = []
    for budget in (148, 5):
        st = make_stage(case, flags=flags)
        st.set_modulation(mod.to(st.device).contiguous())
        y, pool = run_step(st, case, budget)
        err = rel_err(y, y_ref)
        print(f"{name}, sm_budget {budget}: max|err|/RMS = {err:.2e}")
        assert err <= TOL
        outs.append((y, pool))
        if budget == 148:
            st.kv_pool.copy_(wl.bits_to_bf16_tensor(case.kv_pool, st.device))
            st.set_modulation(None)
            y_off, _ = run_step(st, case, budget)
            assert rel_err(y_off, y_plain) <= TOL
        st.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


def test_qkv_bias_argument_errors(orc):
    case = config1_case(orc)
    st = make_stage(case)
    try:
        buf = torch.zeros(1024, dtype=torch.bfloat16, device=st.device)
        for args, code in (((-1, 0, 0, 0), B.HS_ERR_INVALID_ARG), ((1, 0, 0, 0), B.HS_ERR_INVALID_ARG),
                           ((0, buf.data_ptr() + 2, 0, 0), B.HS_ERR_INVALID_ARG)):
            with pytest.raises(B.HsError) as e:
                B.hs_stage_set_qkv_bias(st.handle, *args)
            assert e.value.status == code
        B.hs_stage_set_qkv_bias(st.handle, 0, 0, 0, 0)       # clearing is allowed
    finally:
        st.close()


def test_chunked_prefill_then_decode_on_the_gpu_cache(orc):
    """A multi-step chain that lives on the GPU's own cache: prefill in two chunks, then two decode steps;
    every step is compared with the oracle running the same chain on its own cache."""
    dims = wl.StageDims(2, 256, 4, 2, 64, 688)
    total = wl.BatchSpec([50], [0])
    case = make_case(dims, total, seed=13)
    x_all = wl.make_x(50, dims.d_model, 13)
    st = make_stage(case, max_tokens=64, max_position=64)
    pool_ref = case.kv_pool.copy()
    done = 0
    try:
        for n in (31, 17, 1, 1):
            xs = x_all[done:done + n]
            y_ref = orc.step(case.cfg, case.weights, pool_ref, [n], [done], case.block_tables, wl.to_f32_numpy(xs))
            y, _ = run_step(st, case, 148, q_len=[n], ctx_len=[done], x_t=xs)
            err = rel_err(y, y_ref)
            print(f"chain step n={n} ctx={done}: max|err|/RMS = {err:.2e}")
            assert err <= TOL
            done += n
    finally:
        st.close()


# ------------------------------------------------------ co-run on 2 streams --
def test_corun_on_two_streams_is_bit_identical_to_solo(orc):
    dims_a = wl.StageDims(2, 512, 8, 2, 64, 1408)
    dims_b = wl.StageDims(2, 256, 4, 2, 64, 688)
    case_a = make_case(dims_a, wl.BatchSpec([300, 200, 1, 1], [0, 40, 300, 900]), seed=21, kv_fill=True)
    case_b = make_case(dims_b, wl.BatchSpec([1] * 8, [100 + 90 * i for i in range(8)]), seed=22, kv_fill=True)
    st_a, st_b = make_stage(case_a), make_stage(case_b)
    try:
        ya_solo, pa_solo = run_step(st_a, case_a, 100)
        yb_solo, pb_solo = run_step(st_b, case_b, 48)
        sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
        dev = st_a.device
        xa, xb = case_a.x_t.to(dev), case_b.x_t.to(dev)
        ya = torch.empty(case_a.batch.n_tokens, dims_a.d_model, device=dev)
        yb = torch.empty(case_b.batch.n_tokens, dims_b.d_model, device=dev)
        ba = st_a.make_batch(case_a.batch.q_len, case_a.batch.ctx_len, case_a.block_tables, xa, ya)
        bb = st_b.make_batch(case_b.batch.q_len, case_b.batch.ctx_len, case_b.block_tables, xb, yb)
        torch.cuda.synchronize()
        for _ in range(3):
            st_a.step(ba, 100, sa)
            st_b.step(bb, 48, sb)
        torch.cuda.synchronize()
        assert st_a.status() == 0 and st_b.status() == 0
        assert np.array_equal(ya.cpu().numpy(), ya_solo) and np.array_equal(yb.cpu().numpy(), yb_solo)
        assert np.array_equal(wl.bf16_bits_numpy(st_a.kv_pool).reshape(-1), pa_solo)
        assert np.array_equal(wl.bf16_bits_numpy(st_b.kv_pool).reshape(-1), pb_solo)
        y_ref = orc.step(case_a.cfg, case_a.weights, case_a.kv_pool.copy(), case_a.batch.q_len, case_a.batch.ctx_len,
                         case_a.block_tables, case_a.x)
        assert rel_err(ya_solo, y_ref) <= TOL
    finally:
        st_a.close(); st_b.close()


# ------------------------------------------------------------- SM census --
def test_every_kernel_of_a_step_stays_within_the_sm_budget(orc):
    """Each block records the SM it runs on.  With sm_budget B no kernel class may show more than B
    blocks, and blocks of one launch sit on pairwise different SMs (one block per SM)."""
    dims = wl.StageDims(2, 512, 8, 2, 64, 1408)
    case = make_case(dims, wl.BatchSpec([700, 333, 1, 1, 1, 1], [0, 100, 900, 300, 40, 2000]), seed=41, kv_fill=True)
    st = make_stage(case)
    try:
        st.debug_tensor("smid")                              # switches the census on
        y_ref = None
        for budget in (148, 37, 5, 1):
            y, _ = run_step(st, case, budget)
            census = st.debug_tensor("smid").cpu().numpy()
            used = set()
            for cls, name in enumerate(B.PROFILE_CLASSES):
                sms = census[cls][census[cls] > 0] - 1
                if name == "attn_combine":
                    assert len(sms) == 0
                    continue
                assert 1 <= len(sms) <= budget, (name, budget, len(sms))
                assert len(set(sms.tolist())) == len(sms), (name, budget)      # one block per SM
                used |= set(sms.tolist())
            assert max(used) < st.sm_count
            y_ref = y if y_ref is None else y_ref
            assert np.array_equal(y, y_ref)
    finally:
        st.close()


# ------------------------------------------------- fp16 range of the private activations --
@pytest.mark.parametrize("T", [40, 300])
def test_fp16_saturation_is_counted_and_the_output_stays_finite(orc, T):
    """h, o and act are stored as fp16, clamped to +-65504.  A stage whose SwiGLU activations leave that range
    (gate and up projections scaled x300 here; nothing faults, clamping is defined behaviour) must say so through
    hs_stage_saturation_count and still return finite numbers; the bf16 form of the same stage reports nothing and
    stays within the tolerance.  T = 40 goes through the weight-streaming GEMM, T = 300 through the tiled one."""
    dims = wl.StageDims(1, 512, 8, 2, 64, 1024)
    case = make_case(dims, wl.BatchSpec([T], [0]), seed=41)
    big = [dict(lw) for lw in case.weights_t]
    for k in ("w_gate", "w_up"):
        big[0][k] = (big[0][k].float() * 300.0).to(torch.bfloat16)
    w_np = wl.weights_to_numpy(big)
    y_ref = orc.step(case.cfg, w_np, case.kv_pool.copy(), case.batch.q_len, case.batch.ctx_len, case.block_tables, case.x)
    # the scaled projections of a unit-RMS row have a standard deviation of 0.02 * 300 * sqrt(512) = 136, so
    # silu(gate) * up passes 65504 in the tails; checked on the input rows as a stand-in for the MLP's input
    h_like = orc.rmsnorm(case.x, w_np[0]["g_mlp"], dims.rms_eps)
    assert float(np.max(np.abs(orc.linear(h_like, w_np[0]["w_gate"])))) > 400.0
    st = make_stage(case, weights=big)
    try:
        assert st.saturation_count() == 0
        y, _ = run_step(st, case, st.sm_count, expect_saturation=True)
        n_sat = st.saturation_count()
        assert n_sat > 0, "clamped activations went unreported"
        assert np.all(np.isfinite(y))
        y2, _ = run_step(st, case, 8, expect_saturation=True)
        assert np.array_equal(y, y2)
        assert st.saturation_count() == 2 * n_sat           # the count accumulates, and is the same at every budget
    finally:
        st.close()
    st = make_stage(case, weights=big, flags=B.HS_FLAG_BF16_ACTIVATIONS)
    try:
        y, _ = run_step(st, case, st.sm_count)
        assert st.saturation_count() == 0
        assert rel_err(y, y_ref) <= 3e-2                    # all-bf16 operands: within the format's own floor
    finally:
        st.close()


# ------------------------------------------------- bounded waits --
def test_a_wait_that_nothing_satisfies_gives_up_with_a_timeout_status():
    """The wind-down every kernel runs when a wait exceeds its limit (abort flag, status word, roles leaving, drain,
    tensor memory freed), run on purpose by the probe with a 1 ms limit: it must return by itself with
    HS_ERR_TIMEOUT in the status word, quickly, and leave the context usable for a regular step."""
    import time
    dev = torch.device("cuda:0")
    status = torch.zeros(2, dtype=torch.int32, device=dev)
    waited = torch.zeros(1, dtype=torch.int64, device=dev)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    B.hs_op_wait_probe(1_000_000, status.data_ptr(), waited.data_ptr())
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert status[0].item() == B.HS_ERR_TIMEOUT
    assert 1_000_000 <= waited.item() < 50_000_000          # gave up after the limit, not long after
    assert dt < 1.0
    for bad in (0, 10, 10**9):
        with pytest.raises(B.HsError):
            B.hs_op_wait_probe(bad, status.data_ptr())
    with pytest.raises(B.HsError):
        B.hs_op_wait_probe(1_000_000, 0)
    # the context is intact: a GEMM runs and is right
    a = torch.randn(64, 128, device=dev).to(torch.bfloat16)
    w = torch.randn(256, 128, device=dev).to(torch.bfloat16)
    out = torch.empty(64, 256, device=dev)
    st2 = torch.zeros(1, dtype=torch.int32, device=dev)
    B.hs_op_gemm_bf16(a.data_ptr(), w.data_ptr(), 0, out.data_ptr(), 64, 256, 128, 148, st2.data_ptr())
    torch.cuda.synchronize()
    assert st2.item() == 0
    assert torch.allclose(out, a.float() @ w.float().T, rtol=1e-3, atol=1e-2)


# ------------------------------------------------- RMSNorm folded into the GEMMs --
def test_folded_rmsnorm_step_matches_oracle_and_every_budget(orc):
    """Two layers whose four projections all run on SM pairs, so that both norms of a layer are folded into the GEMMs
    around them (the residual GEMM emits the un-normalised 16-bit operand and the row sums of squares, the next GEMM
    scales its rows): against the oracle on sampled rows, and bit for bit across budgets down to one pair (2) and to
    the single-block stand-in (1), which must add the same partial sums in the same order."""
    dims = wl.StageDims(2, 1024, 16, 4, 64, 2048)
    r = np.random.default_rng(12)
    batch = wl.BatchSpec([1400, 1100] + [1] * 100, [0, 200] + r.integers(30, 900, size=100).tolist())
    case = make_case(dims, batch, seed=77, kv_fill=True)
    rows = np.unique(np.concatenate([np.array([0, 1, 127, 128, 255, 256, 1399, 1400, 2499, 2500, batch.n_tokens - 1]),
                                     np.linspace(0, batch.n_tokens - 1, 60).astype(np.int64)]))
    mask = np.zeros(batch.n_tokens, dtype=np.uint8)
    mask[rows] = 1
    y_ref = orc.step(case.cfg, case.weights, case.kv_pool.copy(), batch.q_len, batch.ctx_len, case.block_tables, case.x,
                     last_layer_row_mask=mask)
    st = make_stage(case)
    try:
        outs = {}
        for budget in (st.sm_count, 37, 2, 1):
            st.kv_pool.copy_(wl.bits_to_bf16_tensor(case.kv_pool, st.device))
            outs[budget] = run_step(st, case, budget)
        y, pool = outs[st.sm_count]
        err = rel_err(y[rows], y_ref[rows])
        print(f"folded RMSNorm, 2 layers, {batch.n_tokens} rows: max|err|/RMS on {len(rows)} rows = {err:.2e}")
        assert err <= TOL
        for budget, (y_b, pool_b) in outs.items():
            assert np.array_equal(y_b, y), budget
            assert np.array_equal(pool_b, pool), budget
        # the fold leaves one RMSNorm launch per step (the first norm, which has no GEMM in front of it)
        B.hs_stage_profile_enable(st.handle, True)
        run_step(st, case, st.sm_count)
        prof = B.hs_stage_profile_read(st.handle)
        B.hs_stage_profile_enable(st.handle, False)
        assert prof["rmsnorm"][1] == 1 and prof["gemm_out"][1] == 2 and prof["gemm_down"][1] == 2
    finally:
        st.close()


@pytest.mark.gpu
@pytest.mark.parametrize("flags", [0, B.HS_FLAG_BF16_ACTIVATIONS])
@pytest.mark.parametrize("n_rows", [16, 9])
def test_small_step_takes_the_norms_into_its_projections(orc, n_rows, flags):
    """Decode-only steps of at most 16 rows: the residual projections on the weight-streaming kernel emit the next
    GEMM's un-normalised 16-bit operand and the rows' sums of squares, the projections behind them scale their output
    rows by the RMSNorm factor, so that a three-layer step launches one RMSNorm (the first, which widens x_in) instead
    of six.  Against the oracle on every row, bit for bit across budgets, in both activation formats."""
    dims = wl.StageDims(3, 1024, 16, 2, 64, 3072)
    r = np.random.default_rng(21)
    batch = wl.BatchSpec([1] * n_rows, r.integers(40, 700, size=n_rows).tolist())
    case = make_case(dims, batch, seed=31, kv_fill=True)
    y_ref = orc.step(case.cfg, case.weights, case.kv_pool.copy(), batch.q_len, batch.ctx_len, case.block_tables, case.x)
    st = make_stage(case, flags=flags)
    try:
        outs = {}
        for budget in (st.sm_count, 40, 3, 1):
            st.kv_pool.copy_(wl.bits_to_bf16_tensor(case.kv_pool, st.device))
            outs[budget] = run_step(st, case, budget)
        y, pool = outs[st.sm_count]
        err = rel_err(y, y_ref)
        print(f"small step with the norms in the projections, {n_rows} rows, flags {flags}: max|err|/RMS = {err:.2e}")
        assert err <= TOL
        for budget, (y_b, pool_b) in outs.items():
            assert np.array_equal(y_b, y), budget
            assert np.array_equal(pool_b, pool), budget
        # the runs above took the one-launch form of the step (after the first norm one cooperative kernel walks all
        # layers, its phases separated by grid barriers); with the per-kernel timers on, the same step runs as one
        # launch per kernel: the same bits, one RMSNorm launch
        B.hs_stage_profile_enable(st.handle, True)
        st.kv_pool.copy_(wl.bits_to_bf16_tensor(case.kv_pool, st.device))
        y_k, pool_k = run_step(st, case, st.sm_count)
        prof = B.hs_stage_profile_read(st.handle)
        B.hs_stage_profile_enable(st.handle, False)
        assert prof["rmsnorm"][1] == 1 and prof["gemm_qkv"][1] == 3 and prof["gemm_gateup"][1] == 3
        assert np.array_equal(y_k, y) and np.array_equal(pool_k, pool)
    finally:
        st.close()


# ------------------------------------------------ guard bytes around every buffer --
GUARDED = {
    # all four projections on SM pairs, both norms folded, stream-K residual GEMMs, both attention kernels side by side
    "pairs_folded": (wl.StageDims(2, 1024, 16, 4, 64, 2048), [1400, 1100] + [1] * 40, [0, 200] + [57 + 13 * i for i in range(40)]),
    # single blocks with a K split, ragged row tile
    "single_blocks": (wl.StageDims(2, 512, 8, 2, 64, 1408), [100, 21, 1], [0, 40, 300]),
    # weight-streaming kernel with the small-step fold
    "small_step": (wl.StageDims(2, 1024, 16, 2, 64, 3072), [1] * 11, [33 + 29 * i for i in range(11)]),
}


@pytest.mark.gpu
@pytest.mark.parametrize("name", sorted(GUARDED))
def test_a_step_writes_nothing_outside_its_buffers(name):
    """Guard bytes in front of and behind the workspace, the KV pool, x_in and y_out keep their pattern through steps
    at several budgets (the step forms differ: SM pairs with folded norms and stream-K, single blocks with a K split,
    the weight-streaming kernel); y_out is written completely."""
    dims, q_len, ctx_len = GUARDED[name]
    batch = wl.BatchSpec(list(q_len), list(ctx_len))
    case = make_case(dims, batch, seed=5, kv_fill=True)
    G = 4096
    st = make_stage(case, guard_bytes=G)
    try:
        T, d = batch.n_tokens, dims.d_model
        x_raw = torch.full((T * d * 2 + 2 * G,), 0xA5, dtype=torch.uint8, device=st.device)
        y_raw = torch.full((T * d * 4 + 2 * G,), 0xA5, dtype=torch.uint8, device=st.device)
        x = x_raw[G: G + T * d * 2].view(torch.bfloat16).view(T, d)
        y = y_raw[G: G + T * d * 4].view(torch.float32).view(T, d)
        x.copy_(case.x_t.to(st.device))
        for budget in (st.sm_count, 37, 2, 1):
            st.kv_pool.copy_(wl.bits_to_bf16_tensor(case.kv_pool, st.device))
            y.fill_(float("nan"))
            st.step(st.make_batch(batch.q_len, batch.ctx_len, case.block_tables, x, y), budget)
            torch.cuda.synchronize()
            assert st.status() == 0
            assert st.guards_intact(), (name, budget)
            for raw in (x_raw, y_raw):
                assert bool((raw[:G] == 0xA5).all()) and bool((raw[-G:] == 0xA5).all()), (name, budget)
            assert bool(torch.isfinite(y).all()), (name, budget)
            assert torch.equal(x, case.x_t.to(st.device)), "x_in is read only"
        # the step forms the cases are named for were the ones that ran
        B.hs_stage_profile_enable(st.handle, True)
        st.step(st.make_batch(batch.q_len, batch.ctx_len, case.block_tables, x, y), st.sm_count)
        torch.cuda.synchronize()
        prof = B.hs_stage_profile_read(st.handle)
        B.hs_stage_profile_enable(st.handle, False)
        assert prof["rmsnorm"][1] == (4 if name == "single_blocks" else 1)
    finally:
        st.close()
