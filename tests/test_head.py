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
