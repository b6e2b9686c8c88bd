"""Brute-force form of the oracle: pure-Python scalar loops, segment by segment.

TEST INFRASTRUCTURE ONLY (tiny inputs).  Written independently of laser_oracle.py as the
literal per-segment statement of the method: for every segment S_i of w consecutive items,
Q = t W_q, K = S_i W_k, V = S_i W_v (Eq. 4) and s_i = Sigmoid(Q K^T / gamma) V (Eq. 5), one
head slice at a time; then for each GSTA layer the explicit projections of every segment
vector, a softmax over the non-empty segments, the weighted sum and the residual (Eq. 7).
The paper states that this iterative form and the global reshaped form give the same result;
tests check the two oracles against each other.  Same readings (heads, masking, ragged tail)
as laser_oracle.py.
"""
from __future__ import annotations

import math


def _sigmoid(x: float) -> float:
    if x >= 0.0:
        return 1.0 / (1.0 + math.exp(-x))
    e = math.exp(x)
    return e / (1.0 + e)


def _vecmat(x, W, n_in, n_out):
    return [sum(float(x[i]) * float(W[i][j]) for i in range(n_in)) for j in range(n_out)]


def sta_one(X, ell, t, Wq, Wk, Wv, S, H, gamma):
    """One user, one candidate: X [L][d], t [d] -> list of L' segment vectors (each a list of d floats)."""
    L, d = len(X), len(t)
    d_qk = len(Wq[0])
    d_qh, d_vh = d_qk // H, d // H
    Lp = -(-L // S)
    q = _vecmat(t, Wq, d, d_qk)                                   # Eq. 4, Q = t W_q
    out = []
    for i in range(Lp):                                           # Eq. 3: segment i = items [iS, (i+1)S)
        s = [0.0] * d
        for n in range(i * S, min((i + 1) * S, L)):
            if n >= ell:
                continue                                          # masked item: contributes nothing
            k = _vecmat(X[n], Wk, d, d_qk)                        # Eq. 4, K row
            v = _vecmat(X[n], Wv, d, d)                           # Eq. 4, V row
            for h in range(H):
                dot = sum(q[h * d_qh + a] * k[h * d_qh + a] for a in range(d_qh))
                g = _sigmoid(dot / gamma)                         # Eq. 5
                for c in range(h * d_vh, (h + 1) * d_vh):
                    s[c] += g * v[c]
        out.append(s)
    return out


def gsta_one(Hp, ell, t, Wg, S, H, tau):
    """One candidate: Hp = list of L' vectors, t [d], Wg [M][3][d][d] -> z (list of d floats)."""
    d = len(t)
    dh = d // H
    Lp = len(Hp)
    n_valid = min(-(-int(ell) // S), Lp)
    tl = [float(x) for x in t]
    if n_valid == 0:
        return tl
    for layer in Wg:
        Wql, Wkl, Wvl = layer[0], layer[1], layer[2]
        q = _vecmat(tl, Wql, d, d)
        ks = [_vecmat(Hp[j], Wkl, d, d) for j in range(n_valid)]
        vs = [_vecmat(Hp[j], Wvl, d, d) for j in range(n_valid)]
        o = [0.0] * d
        for h in range(H):
            sl = range(h * dh, (h + 1) * dh)
            e = [sum(q[c] * ks[j][c] for c in sl) / tau for j in range(n_valid)]
            m = max(e)
            w = [math.exp(x - m) for x in e]
            z = sum(w)
            for j in range(n_valid):
                a = w[j] / z
                for c in sl:
                    o[c] += a * vs[j][c]
        tl = [tl[c] + o[c] for c in range(d)]                     # t_l = t_{l-1} + o_l
    return tl


def forward(items, lengths, cands, cand_offsets, Wq, Wk, Wv, Wg, S, H, gamma, tau):
    """Loops over users and candidates.  Returns (H' as nested lists [N][L'][d], z as [N][d])."""
    Hp_all, z_all = [], []
    for u in range(len(items)):
        for c in range(int(cand_offsets[u]), int(cand_offsets[u + 1])):
            Hp = sta_one(items[u], int(lengths[u]), cands[c], Wq, Wk, Wv, S, H, gamma)
            Hp_all.append(Hp)
            z_all.append(gsta_one(Hp, int(lengths[u]), cands[c], Wg, S, H, tau))
    return Hp_all, z_all
