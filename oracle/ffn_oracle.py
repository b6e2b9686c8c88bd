"""CPU oracle of the feed-forward refinement of the segment vectors (Eq. 6):  s_i <- LN(FFN(s_i) + s_i).

TEST INFRASTRUCTURE ONLY, like the rest of oracle/: imported by tests and the benchmark's checks, never by the CUDA
library or its binding.  float64 numpy, one step per line of the definition.

The paper states the residual + layer-norm form and the expansion ratio r (the cost term 2 r d^2 per segment is two
d x r d matrix products), and nothing else.  Readings taken here (kept identical in the CUDA library):
  * FFN(s) = max(s W_1 + b_1, 0) W_2 + b_2  with W_1 [d, r d], W_2 [r d, d]: the standard two-layer position-wise
    network with a ReLU;
  * LN(y) = (y - mean(y)) / sqrt(var(y) + eps) * g + beta over the d features of one vector, var the biased
    (1/d) variance, eps = 1e-5, with learnable gain g and shift beta;
  * only the vectors of non-empty segments are refined; the zero row of an empty segment stays a zero row (GSTA
    never reads it).

Pins (tests/test_oracle_ffn.py): explicit scalar loops on a tiny case, a hand-computed layer norm, torch's
linear / relu / layer_norm on the valid rows, the zero-FFN case (output = LN(s)), a case whose hidden units are all
switched off by the ReLU (output = LN(s + b_2)), mean / variance invariants of the normalised output, and checks
that a dropped residual, a transposed weight or an unbiased variance would be caught.
"""
from __future__ import annotations

import numpy as np

LN_EPS = 1e-5


def layer_norm(y, g, beta, eps=LN_EPS):
    """Layer norm over the last axis: biased variance, gain g, shift beta."""
    y = np.asarray(y, dtype=np.float64)
    mean = y.mean(axis=-1, keepdims=True)
    var = ((y - mean) ** 2).mean(axis=-1, keepdims=True)
    return (y - mean) / np.sqrt(var + eps) * np.asarray(g, dtype=np.float64) + np.asarray(beta, dtype=np.float64)


def ffn_rows(s, W1, b1, W2, b2, g, beta, eps=LN_EPS):
    """Eq. 6 on rows: s [..., d] -> LN(max(s W1 + b1, 0) W2 + b2 + s)."""
    s = np.asarray(s, dtype=np.float64)
    W1, b1, W2, b2 = (np.asarray(a, dtype=np.float64) for a in (W1, b1, W2, b2))
    hidden = np.maximum(s @ W1 + b1, 0.0)
    y = hidden @ W2 + b2 + s
    return layer_norm(y, g, beta, eps)


def ffn_forward(Hp, lengths, cand_offsets, S, W1, b1, W2, b2, g, beta, eps=LN_EPS):
    """Eq. 6 over the compact sequences.  Hp [N, L', d]; the rows of each candidate's non-empty segments are refined,
    the others stay zero.  Returns [N, L', d] float64."""
    Hp = np.asarray(Hp, dtype=np.float64)
    N, Lp, d = Hp.shape
    out = np.zeros_like(Hp)
    for u in range(len(lengths)):
        a, b = int(cand_offsets[u]), int(cand_offsets[u + 1])
        n = min(-(-int(lengths[u]) // int(S)), Lp)
        if b > a and n > 0:
            out[a:b, :n] = ffn_rows(Hp[a:b, :n], W1, b1, W2, b2, g, beta, eps)
    return out
