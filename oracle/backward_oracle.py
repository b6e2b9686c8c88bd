"""CPU oracle for the backward pass of LASER's STA + GSTA forward (the vector-Jacobian product of z).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's parity / CPU-baseline legs, never
by the product path; it shares no code with the CUDA sources.

The paper trains the model (section "Experimental Settings") but prints no backward formulas: the definition is the
derivative of the forward map of `laser_oracle.py` (Eq. 8-12, then Eq. 7 with the residual update).  Given the upstream
gradient dz = dLoss/dz [N, d], this file returns dLoss/d(every input): items, candidates, W_q, W_k, W_v and the GSTA
weights, in float64, by the chain rule written out step by step in the reverse order of the forward:

  GSTA layer l = M .. 1   t_l = t_{l-1} + o_l,  o = a v,  a = softmax_j(q . k_j / tau),  q = t_{l-1} W_q^l,
                          k_j = s_j W_k^l,  v_j = s_j W_v^l                                              (Eq. 7)
        do = dt_l;  da_j = do . v_j;  dv_j = a_j do;  de_j = a_j (da_j - sum_i a_i da_i) / tau;
        dq = sum_j de_j k_j;  dk_j = de_j q;  ds_j += dk_j W_k^T + dv_j W_v^T;  dt_{l-1} = dt_l + dq W_q^T
  STA                     s_i[head h] = sum_{n in segment i, n < len} alpha_{n,h} v_{n,h},  alpha = Sigmoid(q_h . k_{n,h} / gamma)
                                                                                                          (Eq. 10-12)
        dalpha_{n,h} = ds_i[h] . v_{n,h};  dv_{n,h} += alpha_{n,h} ds_i[h];
        dscore = dalpha alpha (1 - alpha) / gamma;  dq_h += dscore k_{n,h};  dk_{n,h} += dscore q_h
  projections             Q = T W_q, K = X W_k, V = X W_v                                                 (Eq. 8-9)

Readings are those of the forward oracle: an item at or past `len` has gate 0 (so it receives and passes no gradient:
its row of d_items is exactly zero), an empty segment is outside the GSTA softmax (no gradient reaches it).

Pins (tests/test_oracle_backward.py): central finite differences of sum(dz * z) through `laser_oracle.forward` on every
input, torch.autograd through an independent per-segment restatement of the forward, M = 0 (dz passes straight to the
candidates), linearity in dz, zero rows for padding, invariance to the padded rows' contents.
"""
from __future__ import annotations

import numpy as np
from scipy.special import expit

from .laser_oracle import default_gamma, default_tau, num_segments


def backward_user(X, ell, T, Wq, Wk, Wv, Wg, S, H, gamma, tau, dz):
    """One user: X [L, d], T [C, d], dz [C, d] -> (dX [L, d], dT [C, d], dWq, dWk, dWv, dWg) float64."""
    X = np.asarray(X, dtype=np.float64)
    T = np.asarray(T, dtype=np.float64)
    Wq, Wk, Wv, Wg = (np.asarray(w, dtype=np.float64) for w in (Wq, Wk, Wv, Wg))
    dz = np.asarray(dz, dtype=np.float64)
    L, d = X.shape
    C = T.shape[0]
    d_qk = Wq.shape[1]
    d_qh, d_vh = d_qk // H, d // H
    M = Wg.shape[0]
    Lp = num_segments(L, S)
    ell = int(ell)

    # ---- forward, keeping what the backward needs
    Q = T @ Wq
    K = X @ Wk
    V = X @ Wv
    Qh = Q.reshape(C, H, d_qh)
    Kh = K.reshape(L, H, d_qh)
    valid = (np.arange(L) < ell)
    sig = expit(np.einsum("chq,nhq->chn", Qh, Kh) / gamma)          # [C, H, L]
    alpha = sig * valid[None, None, :]
    pad = Lp * S - L
    alpha_p = np.concatenate([alpha, np.zeros((C, H, pad))], axis=2) if pad else alpha
    V_p = np.concatenate([V, np.zeros((pad, d))], axis=0) if pad else V
    A_hat = alpha_p.reshape(C, H, Lp, S)
    V_hat = V_p.reshape(Lp, S, H, d_vh)
    Hp = np.einsum("chiw,iwhv->cihv", A_hat, V_hat).reshape(C, Lp, d)
    nv = min(num_segments(ell, S), Lp) if ell > 0 else 0
    Hv = Hp[:, :nv, :]
    t_prev, qs, ks, vs, attn = [], [], [], [], []
    t = T.copy()
    if nv > 0:
        for l in range(M):
            q = (t @ Wg[l, 0]).reshape(C, H, d_vh)
            k = (Hv @ Wg[l, 1]).reshape(C, nv, H, d_vh)
            v = (Hv @ Wg[l, 2]).reshape(C, nv, H, d_vh)
            e = np.einsum("chx,cjhx->chj", q, k) / tau
            e = e - e.max(axis=2, keepdims=True)
            a = np.exp(e)
            a = a / a.sum(axis=2, keepdims=True)
            t_prev.append(t)
            qs.append(q); ks.append(k); vs.append(v); attn.append(a)
            t = t + np.einsum("chj,cjhx->chx", a, v).reshape(C, d)

    # ---- backward through the GSTA layers, last to first
    dWg = np.zeros_like(Wg)
    dt = dz.copy()
    dHv = np.zeros((C, nv, d))
    if nv > 0:
        for l in reversed(range(M)):
            q, k, v, a = qs[l], ks[l], vs[l], attn[l]
            do = dt.reshape(C, H, d_vh)
            da = np.einsum("chx,cjhx->chj", do, v)
            dv = np.einsum("chj,chx->cjhx", a, do)
            de = a * (da - (a * da).sum(axis=2, keepdims=True)) / tau
            dq = np.einsum("chj,cjhx->chx", de, k).reshape(C, d)
            dk = np.einsum("chj,chx->cjhx", de, q).reshape(C, nv, d)
            dv = dv.reshape(C, nv, d)
            dWg[l, 1] += np.einsum("cjd,cje->de", Hv, dk)
            dWg[l, 2] += np.einsum("cjd,cje->de", Hv, dv)
            dHv += dk @ Wg[l, 1].T + dv @ Wg[l, 2].T
            dWg[l, 0] += t_prev[l].T @ dq
            dt = dt + dq @ Wg[l, 0].T
    dT = dt                                                          # through t_0 = T; the path through Q is added below

    # ---- backward through the segment aggregation and the gates
    dHp4 = np.zeros((C, Lp, H, d_vh))
    dHp4[:, :nv] = dHv.reshape(C, nv, H, d_vh)
    dA_hat = np.einsum("cihv,iwhv->chiw", dHp4, V_hat)
    dV_hat = np.einsum("chiw,cihv->iwhv", A_hat, dHp4)
    dalpha = dA_hat.reshape(C, H, Lp * S)[:, :, :L] * valid[None, None, :]
    dV = dV_hat.reshape(Lp * S, d)[:L]
    dscore = dalpha * sig * (1.0 - sig) / gamma
    dQ = np.einsum("chn,nhq->chq", dscore, Kh).reshape(C, d_qk)
    dK = np.einsum("chn,chq->nhq", dscore, Qh).reshape(L, d_qk)

    # ---- backward through the projections
    dWq = T.T @ dQ
    dWk = X.T @ dK
    dWv = X.T @ dV
    dT = dT + dQ @ Wq.T
    dX = dK @ Wk.T + dV @ Wv.T
    return dX, dT, dWq, dWk, dWv, dWg


def backward(items, lengths, cands, cand_offsets, Wq, Wk, Wv, Wg, S, H, dz, gamma=None, tau=None, users=None):
    """Batched.  Returns a dict of float64 arrays: d_items [U, L, d], d_cands [N, d], dWq, dWk, dWv, dWg.
    `users` restricts the work to some users (the others contribute nothing: their rows stay zero)."""
    items = np.asarray(items)
    U, L, d = items.shape
    N = int(cand_offsets[-1])
    if gamma is None or gamma <= 0:
        gamma = default_gamma(np.shape(Wq)[1], H)
    if tau is None or tau <= 0:
        tau = default_tau(d, H)
    out = {"d_items": np.zeros((U, L, d)), "d_cands": np.zeros((N, d)), "dWq": np.zeros(np.shape(Wq)),
           "dWk": np.zeros(np.shape(Wk)), "dWv": np.zeros(np.shape(Wv)), "dWg": np.zeros(np.shape(Wg))}
    for u in (range(U) if users is None else users):
        a, b = int(cand_offsets[u]), int(cand_offsets[u + 1])
        if b <= a:
            continue
        dX, dT, dWq, dWk, dWv, dWg = backward_user(items[u], lengths[u], cands[a:b], Wq, Wk, Wv, Wg, S, H, gamma, tau,
                                                   np.asarray(dz)[a:b])
        out["d_items"][u] = dX
        out["d_cands"][a:b] = dT
        out["dWq"] += dWq
        out["dWk"] += dWk
        out["dWv"] += dWv
        out["dWg"] += dWg
    return out
