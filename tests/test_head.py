"""The ends of the stage: embedding, final RMSNorm + vocabulary projection + greedy sampling.

CPU part: pins of the oracle.  GPU part (marked): the library's kernels against the oracle."""
import numpy as np
import pytest
import torch

from oracle import head as OH
from oracle.oracle import Oracle
from paper_2608_01785_b200 import workloads as wl
from tests.helpers import rel_err


@pytest.fixture(scope="module")
def orc():
    return Oracle("f32")


# ------------------------------------------------------------------ oracle pins --
def test_argmax_is_the_first_maximum_and_matches_the_library_routine():
    rng = np.random.default_rng(0)
    a = rng.standard_normal((7, 300)).astype(np.float32)
    assert np.array_equal(OH.argmax_first(a), np.argmax(a, axis=1))
    assert np.array_equal(OH.argmax_first(a + 5.0), OH.argmax_first(a))          # shift invariance
    t = np.zeros((3, 10), dtype=np.float32)
    t[0, [4, 7]] = 2.0                                                           # tie: the lower index wins
    t[1, :] = -1.0                                                               # all equal: index 0
    t[2, 9] = 1e-30
    assert OH.argmax_first(t).tolist() == [4, 0, 9]
    assert np.argmax(t, axis=1).tolist() == [4, 0, 9]                            # the routine head() relies on


def test_embed_copies_rows_bit_for_bit():
    table = np.arange(50 * 8, dtype=np.uint16).reshape(50, 8)
    out = OH.embed(table, [3, 3, 49, 0])
    assert out.tolist() == [table[3].tolist(), table[3].tolist(), table[49].tolist(), table[0].tolist()]
    with pytest.raises(AssertionError):
        OH.embed(table, [50])


def test_head_closed_forms(orc):
    d, V = 64, 40
    rng = np.random.default_rng(1)
    y = rng.standard_normal((9, d)).astype(np.float32)
    g = np.ones(d, dtype=np.float32)
    # one-hot vocabulary rows: logit v is the normalised coordinate v, so the sampled token is argmax |.|-free
    w = np.zeros((V, d), dtype=np.float32)
    w[np.arange(V), np.arange(V)] = 1.0
    logits, tok = OH.head(orc, y, [8, 0, 3], g, w, 1e-6)
    for r, src in enumerate([8, 0, 3]):
        norm = y[src] / np.sqrt(np.mean(y[src].astype(np.float64) ** 2) + 1e-6)
        assert np.allclose(logits[r], norm[:V], rtol=1e-5, atol=1e-6)
        assert tok[r] == int(np.argmax(y[src, :V]))
    # scaling a row does not change its token (RMSNorm removes the scale); negating w_vocab gives the argmin
    _, tok2 = OH.head(orc, 7.5 * y, [8, 0, 3], g, w, 1e-12)
    assert np.array_equal(tok, tok2)
    _, tok3 = OH.head(orc, y, [8, 0, 3], g, -w, 1e-6)
    assert tok3.tolist() == [int(np.argmin(y[s, :V])) for s in (8, 0, 3)]


# -------------------------------------------------------------- library on the GPU --
def _head_case(d, V, T, n, seed):
    g = torch.Generator().manual_seed(seed)
    y = torch.randn(T, d, generator=g)
    gain = (1.0 + 0.02 * torch.randn(d, generator=g)).to(torch.bfloat16)
    w = (0.02 * torch.randn(V, d, generator=g)).to(torch.bfloat16)
    rows = torch.randperm(T, generator=g)[:n].to(torch.int32)
    return y, gain, w, rows


@pytest.mark.gpu
@pytest.mark.parametrize("d,V,T,n", [(256, 1000, 50, 7), (1024, 32008, 300, 64), (512, 4104, 128, 128)])
def test_head_step_matches_oracle_and_is_budget_invariant(orc, d, V, T, n):
    from paper_2608_01785_b200 import binding as B
    dev = torch.device("cuda:0")
    y, gain, w, rows = _head_case(d, V, T, n, seed=d + n)
    logits_ref, tok_ref = OH.head(orc, y.numpy(), rows.numpy(), gain.float().numpy(), w.float().numpy(), 1e-6)
    cfg = B.make_head_config(d, V, 1e-6, 128)
    ws = torch.empty(B.hs_head_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
    y_d, gain_d, w_d, rows_d = y.to(dev), gain.to(dev), w.to(dev), rows.to(dev)
    head = B.hs_head_create(cfg, gain_d.data_ptr(), w_d.data_ptr(), ws.data_ptr())
    try:
        outs = []
        for budget in (148, 37, 3):
            logits = torch.full((n, V), float("nan"), device=dev)
            tokens = torch.full((n,), -1, dtype=torch.int32, device=dev)
            B.hs_head_step(head, y_d.data_ptr(), rows_d.data_ptr(), n, logits.data_ptr(), tokens.data_ptr(), budget)
            torch.cuda.synchronize()
            assert B.hs_head_status(head) == B.HS_OK
            outs.append((logits.cpu().numpy(), tokens.cpu().numpy()))
        lg, tk = outs[0]
        for other in outs[1:]:
            assert np.array_equal(other[0], lg) and np.array_equal(other[1], tk)
        err = rel_err(lg, logits_ref)
        print(f"head d={d} V={V} n={n}: logits max|err|/RMS = {err:.2e}")
        assert np.all(np.isfinite(lg)) and err <= 2e-2
        # the sampled token is the first maximum of the GPU's own logits (same precision on both sides) ...
        assert np.array_equal(tk, np.argmax(lg, axis=1).astype(np.int32))
        # ... and the oracle's token wherever the oracle's best two logits are further apart than the error
        top2 = np.sort(logits_ref, axis=1)[:, -2:]
        clear = (top2[:, 1] - top2[:, 0]) > 2 * np.max(np.abs(lg - logits_ref))
        assert clear.sum() >= n // 2 and np.array_equal(tk[clear], tok_ref[clear])
    finally:
        B.hs_head_destroy(head)


@pytest.mark.gpu
def test_argmax_takes_the_lowest_index_on_ties():
    """Logits with exact ties: a zero vocabulary matrix gives all-zero logits (token 0); duplicated vocabulary
    rows give pairs of equal logits (the lower of the two wins)."""
    from paper_2608_01785_b200 import binding as B
    dev = torch.device("cuda:0")
    d, V, n = 128, 2048, 5
    y, gain, w, rows = _head_case(d, V, 20, n, seed=9)
    w[1024:] = w[:1024]                                           # row v + 1024 duplicates row v
    cfg = B.make_head_config(d, V, 1e-6, 8)
    ws = torch.empty(B.hs_head_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
    for weights, check in ((w, lambda t: bool((t < 1024).all())), (torch.zeros_like(w), lambda t: bool((t == 0).all()))):
        y_d, gain_d, w_d, rows_d = y.to(dev), gain.to(dev), weights.to(dev), rows.to(dev)
        head = B.hs_head_create(cfg, gain_d.data_ptr(), w_d.data_ptr(), ws.data_ptr())
        logits = torch.empty(n, V, device=dev)
        tokens = torch.empty(n, dtype=torch.int32, device=dev)
        B.hs_head_step(head, y_d.data_ptr(), rows_d.data_ptr(), n, logits.data_ptr(), tokens.data_ptr(), 148)
        torch.cuda.synchronize()
        B.hs_head_destroy(head)
        assert check(tokens.cpu())
        assert np.array_equal(tokens.cpu().numpy(), np.argmax(logits.cpu().numpy(), axis=1))


@pytest.mark.gpu
def test_embed_copies_rows_and_flags_bad_ids():
    from paper_2608_01785_b200 import binding as B
    dev = torch.device("cuda:0")
    V, d, n = 5000, 1032, 777
    g = torch.Generator().manual_seed(2)
    table = torch.randn(V, d, generator=g).to(torch.bfloat16)
    tokens = torch.randint(0, V, (n,), generator=g, dtype=torch.int32)
    want = OH.embed(wl.bf16_bits_numpy(table), tokens.numpy())
    table_d, tok_d = table.to(dev), tokens.to(dev)
    for budget in (148, 2):
        x = torch.full((n, d), float("nan"), dtype=torch.bfloat16, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        B.hs_op_embed(tok_d.data_ptr(), n, table_d.data_ptr(), V, d, x.data_ptr(), budget, status.data_ptr())
        torch.cuda.synchronize()
        assert status.item() == 0 and np.array_equal(wl.bf16_bits_numpy(x.cpu()), want)      # bit for bit
    bad = tokens.clone()
    bad[5], bad[600] = V, -1
    x = torch.full((n, d), float("nan"), dtype=torch.bfloat16, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    B.hs_op_embed(bad.to(dev).data_ptr(), n, table_d.data_ptr(), V, d, x.data_ptr(), 148, status.data_ptr())
    torch.cuda.synchronize()
    got = wl.bf16_bits_numpy(x.cpu())
    assert status.item() == B.HS_ERR_INVALID_ARG and not got[5].any() and not got[600].any()
    keep = np.ones(n, dtype=bool)
    keep[[5, 600]] = False
    assert np.array_equal(got[keep], want[keep])
    with pytest.raises(B.HsError):
        B.hs_op_embed(tok_d.data_ptr(), n, table_d.data_ptr(), V, 12, x.data_ptr(), 148, status.data_ptr())   # d % 8


def test_head_configuration_errors_on_the_host():
    from paper_2608_01785_b200 import binding as B
    assert B.hs_head_workspace_bytes(B.make_head_config(1024, 32000, 1e-6, 64)) >= 64 * 1024 * 2
    for cfg in (B.make_head_config(1020, 32000, 1e-6, 64), B.make_head_config(1024, 32001, 1e-6, 64),
                B.make_head_config(1024, 32000, 1e-6, 129), B.make_head_config(1024, 32000, 1e-6, 0)):
        assert B.hs_head_workspace_bytes(cfg) == 0
        with pytest.raises(B.HsError):
            B.hs_head_create(cfg, 16, 16, 256)
