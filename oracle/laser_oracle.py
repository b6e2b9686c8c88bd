"""CPU oracle for LASER's Segmented Target Attention + Global Stacked Target Attention forward.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain float64 definition that the
CUDA library is checked against; it is imported only by the tests, the smoke check and
the benchmark's CPU-baseline leg, never by the product path, and it shares no code with
the CUDA sources.

Everything is the paper's definition written out with numpy in float64, in the paper's
"global" (vectorised) order of operations:

  * Q = t W_q, K = H W_k, V = H W_v over the whole sequence           (Eq. 8, Eq. 9)
  * alpha = Sigmoid(Q K^T / gamma), one independent gate per item      (Eq. 10; Eq. 5)
  * reshape alpha and V to (L' x w) windows and batch-multiply         (Eq. 11, Eq. 12)
  * GSTA: per layer a single-query softmax attention of the target over the L' segment
    vectors, a_l = softmax((t_{l-1} W_q^l)(H' W_k^l)^T / scale), o_l = a_l (H' W_v^l),
    followed by t_l = t_{l-1} + o_l                                      (Eq. 7)

Readings where the paper is silent (kept identical in the CUDA library):
  * heads: W_q, W_k are [d, H*d_qh], W_v and the GSTA weights are [d, d]; columns are split
    into H contiguous slices, each head gates / attends on its own slice, head outputs are
    concatenated, and there is no output projection (the experiment section only says
    "2 heads, d_q 16 per head, value dimension d").
  * ragged sequences: the valid items of a user are the prefix [0, len); an item at or past
    len contributes exactly nothing (its gate is forced to 0, not Sigmoid(0)); a segment with
    no valid item gives a zero vector and is left out of the GSTA softmax; len = 0 gives
    H' = 0 and z = t.
  * L not a multiple of the segment size: L' = ceil(L / w), the last segment is short.
  * no FFN / LayerNorm between the two stages (Eq. 6 is outside this path), no biases.
  * GSTA scale: sqrt(d / H) by default (equals the paper's sqrt(d) for one head).

Pins (tests/test_oracle_*.py): brute-force per-segment loops of Eq. 4-5 and Eq. 7, the
one-segment closed form, the all-gates-one-half sum-pooling case, saturation limits,
scaled_dot_product_attention for the GSTA layer, masking / permutation / linearity /
independence invariants.  The paper prints no worked numerical example of s_i, H' or z, so
the values on the five benchmark configurations themselves are "parity unpinned" beyond
those definition-level checks.
"""
from __future__ import annotations

import math

import numpy as np
from scipy.special import expit


def num_segments(L: int, S: int) -> int:
    return -(-int(L) // int(S))


def default_gamma(d_qk: int, H: int) -> float:
    return math.sqrt(d_qk / H)


def default_tau(d: int, H: int) -> float:
    return math.sqrt(d / H)


def sta_user(X, ell, T, Wq, Wk, Wv, S, H, gamma):
    """STA for one user: X [L, d] items (rows >= ell are padding), T [C, d] candidates -> H' [C, L', d].

    Global form, Eq. 8-12: project the whole sequence once, gate every (candidate, item, head),
    zero the gates of masked items, reshape to windows of S items and sum gate * value per window.
    """
    X = np.asarray(X, dtype=np.float64)
    T = np.asarray(T, dtype=np.float64)
    Wq, Wk, Wv = (np.asarray(w, dtype=np.float64) for w in (Wq, Wk, Wv))
    L, d = X.shape
    C = T.shape[0]
    d_qk, d_v = Wq.shape[1], Wv.shape[1]          # d_v = d in the paper; kept general for head-slice checks
    assert d_v % H == 0 and d_qk % H == 0
    d_qh, d_vh = d_qk // H, d_v // H
    Lp = num_segments(L, S)

    Q = T @ Wq                                    # Eq. 8   [C, d_qk]
    K = X @ Wk                                    # Eq. 9   [L, d_qk]
    V = X @ Wv                                    # Eq. 9   [L, d]

    Qh = Q.reshape(C, H, d_qh)
    Kh = K.reshape(L, H, d_qh)
    scores = np.einsum("chq,nhq->chn", Qh, Kh) / gamma   # [C, H, L]
    alpha = expit(scores)                                 # Eq. 10
    valid = (np.arange(L) < int(ell))
    alpha = alpha * valid[None, None, :]                  # masked items contribute nothing

    # R(.): pad L up to L'*S with zero gates / zero values, reshape to windows   (Eq. 11)
    pad = Lp * S - L
    if pad:
        alpha = np.concatenate([alpha, np.zeros((C, H, pad))], axis=2)
        V = np.concatenate([V, np.zeros((pad, d_v))], axis=0)
    A_hat = alpha.reshape(C, H, Lp, S)
    V_hat = V.reshape(Lp, S, H, d_vh)
    Hp = np.einsum("chiw,iwhv->cihv", A_hat, V_hat)       # Eq. 12, batched over windows
    return Hp.reshape(C, Lp, d_v)


def gsta_user(Hp, ell, T, Wg, S, H, tau):
    """GSTA for one user: Hp [C, L', d] segment vectors per candidate, T [C, d] -> z [C, d]   (Eq. 7).

    Every layer attends to the same H' with its own (W_q^l, W_k^l, W_v^l); only the target is updated.
    """
    Hp = np.asarray(Hp, dtype=np.float64)
    t = np.asarray(T, dtype=np.float64).copy()
    Wg = np.asarray(Wg, dtype=np.float64)
    C, Lp, d = Hp.shape
    M = Wg.shape[0]
    assert d % H == 0
    dh = d // H
    n_valid = min(num_segments(int(ell), S), Lp) if int(ell) > 0 else 0
    if n_valid == 0:
        return t
    Hv = Hp[:, :n_valid, :]                               # non-empty segments only
    for l in range(M):
        Wql, Wkl, Wvl = Wg[l, 0], Wg[l, 1], Wg[l, 2]
        q = (t @ Wql).reshape(C, H, dh)
        k = (Hv @ Wkl).reshape(C, n_valid, H, dh)
        v = (Hv @ Wvl).reshape(C, n_valid, H, dh)
        e = np.einsum("chx,cjhx->chj", q, k) / tau
        e = e - e.max(axis=2, keepdims=True)
        a = np.exp(e)
        a = a / a.sum(axis=2, keepdims=True)
        o = np.einsum("chj,cjhx->chx", a, v).reshape(C, d)
        t = t + o
    return t


def sta_forward(items, lengths, cands, cand_offsets, Wq, Wk, Wv, S, H, gamma=None):
    """Batched STA.  items [U, L, d], lengths [U], cands [N, d], cand_offsets [U+1] -> H' [N, L', d] float64."""
    U, L, d = items.shape
    N = int(cand_offsets[-1])
    Lp = num_segments(L, S)
    if gamma is None or gamma <= 0:
        gamma = default_gamma(np.shape(Wq)[1], H)
    out = np.zeros((N, Lp, np.shape(Wv)[1]), dtype=np.float64)
    for u in range(U):
        a, b = int(cand_offsets[u]), int(cand_offsets[u + 1])
        if b > a:
            out[a:b] = sta_user(items[u], lengths[u], cands[a:b], Wq, Wk, Wv, S, H, gamma)
    return out


def gsta_forward(Hp, lengths, cand_offsets, cands, Wg, S, H, tau=None):
    """Batched GSTA.  Hp [N, L', d], cands [N, d], Wg [M, 3, d, d] -> z [N, d] float64."""
    N, Lp, d = np.shape(Hp)
    if tau is None or tau <= 0:
        tau = default_tau(d, H)
    z = np.zeros((N, d), dtype=np.float64)
    for u in range(len(lengths)):
        a, b = int(cand_offsets[u]), int(cand_offsets[u + 1])
        if b > a:
            z[a:b] = gsta_user(Hp[a:b], lengths[u], cands[a:b], Wg, S, H, tau)
    return z


def forward(items, lengths, cands, cand_offsets, Wq, Wk, Wv, Wg, S, H, gamma=None, tau=None,
            users=None, return_hprime=True):
    """STA followed by GSTA.  Returns (H' [N, L', d] or None, z [N, d]); `users` restricts the work to an
    iterable of user indices (rows of other users' candidates are left zero)."""
    U, L, d = items.shape
    N = int(cand_offsets[-1])
    Lp = num_segments(L, S)
    if gamma is None or gamma <= 0:
        gamma = default_gamma(np.shape(Wq)[1], H)
    if tau is None or tau <= 0:
        tau = default_tau(d, H)
    Hp_all = np.zeros((N, Lp, d), dtype=np.float64) if return_hprime else None
    z = np.zeros((N, d), dtype=np.float64)
    for u in (range(U) if users is None else users):
        a, b = int(cand_offsets[u]), int(cand_offsets[u + 1])
        if b <= a:
            continue
        Hp = sta_user(items[u], lengths[u], cands[a:b], Wq, Wk, Wv, S, H, gamma)
        z[a:b] = gsta_user(Hp, lengths[u], cands[a:b], Wg, S, H, tau)
        if return_hprime:
            Hp_all[a:b] = Hp
    return Hp_all, z
