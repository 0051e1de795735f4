"""Oracle of the two ends of the stage (TEST INFRASTRUCTURE ONLY): token embedding in front of the step, and
behind it the final RMSNorm, the vocabulary projection and greedy sampling on the last row of each sequence.

The paper keeps its runtime's model execution unchanged (Sec. 5) and prints nothing for these; they are the
textbook definitions, composed from the oracle's pinned primitives (rmsnorm, linear):
    x[t, :]      = E[token[t], :]                                   (a copy of bf16 rows)
    h[r, :]      = rmsnorm(y[row[r], :]; g_final)                   (fp32)
    logits[r, v] = sum_i h[r, i] * W_vocab[v, i]                    (fp32)
    token[r]     = the lowest v that attains max_v logits[r, v]     (greedy sampling)

Parity status: no worked example in the paper (paper-level parity unpinned); argmax is pinned by a brute-force
loop, its tie rule and shift invariance, the rest by the pins of rmsnorm and linear.
"""
from __future__ import annotations

import numpy as np

from .oracle import Oracle


def embed(table_bits: np.ndarray, tokens) -> np.ndarray:
    """table_bits: uint16 [V, d] (bf16 bit patterns); returns uint16 [n, d]."""
    tokens = np.asarray(tokens, dtype=np.int64)
    assert tokens.min() >= 0 and tokens.max() < table_bits.shape[0]
    return table_bits[tokens].copy()


def argmax_first(logits: np.ndarray) -> np.ndarray:
    """Row-wise index of the maximum; the lowest index on ties.  Written as the plain scan."""
    out = np.zeros(logits.shape[0], dtype=np.int32)
    for r in range(logits.shape[0]):
        best, best_v = 0, logits[r, 0]
        for v in range(1, logits.shape[1]):
            if logits[r, v] > best_v:
                best, best_v = v, logits[r, v]
        out[r] = best
    return out


def head(orc: Oracle, y: np.ndarray, rows, g_final: np.ndarray, w_vocab: np.ndarray, eps: float):
    """y: [T, d]; rows: indices of the rows to sample from; returns (logits [n, V], tokens [n])."""
    sel = np.ascontiguousarray(np.asarray(y, dtype=orc.dtype)[np.asarray(rows, dtype=np.int64)])
    h = orc.rmsnorm(sel, g_final, eps)
    logits = orc.linear(h, w_vocab)
    return logits, np.argmax(logits, axis=1).astype(np.int32)     # numpy's argmax returns the first maximum
