"""CPU oracle of the softmax-aggregation variant of Segmented Target Attention (the paper's ablation of the sigmoid gate).

TEST INFRASTRUCTURE ONLY, like the rest of oracle/: imported by tests, never by the CUDA library or its binding.

The component-ablation study swaps the sigmoid aggregation of Eq. 5 for an ordinary softmax: inside every segment the
weights of the items are normalised to sum to one.  Written out, per candidate t, segment i and head h, over the valid
items n of the segment,

    a_n = exp(q_h . k_{n,h} / gamma) / sum_m exp(q_h . k_{m,h} / gamma),      s_i[head h] = sum_n a_n v_{n,h}

with q, k, v the projections of Eq. 4.  Readings (kept identical in the CUDA library): the heads, the ragged-length
rules and gamma are those of the sigmoid path; the normalisation runs over the valid items of the segment only; a
segment without valid items gives a zero vector.

Pins (tests/test_oracle_softmax_sta.py): scalar loops, scipy's softmax, W_q = 0 (mean pooling of the values), one-item
segments (s = v), the hard-attention limit gamma -> 0, convex-hull and shift invariances, padding irrelevance.
"""
from __future__ import annotations

import numpy as np


def sta_softmax_user(X, ell, T, Wq, Wk, Wv, S, H, gamma):
    """One user: X [L, d] items (rows >= ell are padding), T [C, d] candidates -> H' [C, L', d] float64."""
    X = np.asarray(X, dtype=np.float64)
    T = np.asarray(T, dtype=np.float64)
    Wq, Wk, Wv = (np.asarray(w, dtype=np.float64) for w in (Wq, Wk, Wv))
    L, d = X.shape
    C = T.shape[0]
    d_qk, d_v = Wq.shape[1], Wv.shape[1]
    d_qh, d_vh = d_qk // H, d_v // H
    Lp = -(-L // int(S))
    Q = (T @ Wq).reshape(C, H, d_qh)
    K = (X @ Wk).reshape(L, H, d_qh)
    V = (X @ Wv).reshape(L, H, d_vh)
    out = np.zeros((C, Lp, H, d_vh), dtype=np.float64)
    for i in range(Lp):
        n0, n1 = i * S, min((i + 1) * S, L, int(ell))
        if n1 <= n0:
            continue
        e = np.einsum("chq,nhq->chn", Q, K[n0:n1]) / gamma          # [C, H, items of the segment]
        e = e - e.max(axis=2, keepdims=True)
        a = np.exp(e)
        a = a / a.sum(axis=2, keepdims=True)
        out[:, i] = np.einsum("chn,nhv->chv", a, V[n0:n1])
    return out.reshape(C, Lp, d_v)


def sta_softmax_forward(items, lengths, cands, cand_offsets, Wq, Wk, Wv, S, H, gamma):
    """Batched.  items [U, L, d], cands [N, d] -> H' [N, L', d] float64."""
    U, L, d = items.shape
    N = int(cand_offsets[-1])
    out = np.zeros((N, -(-L // int(S)), np.shape(Wv)[1]), dtype=np.float64)
    for u in range(U):
        a, b = int(cand_offsets[u]), int(cand_offsets[u + 1])
        if b > a:
            out[a:b] = sta_softmax_user(items[u], lengths[u], cands[a:b], Wq, Wk, Wv, S, H, gamma)
    return out
