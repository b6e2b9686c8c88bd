"""Pins for the CPU oracle: everything here checks oracle/ against something other than itself
(brute-force loops of the per-segment definition, closed forms, library attention, invariants)."""
import math
import os

import numpy as np
import pytest
from scipy.special import softmax as sp_softmax

from oracle import cost_model, laser_brute, laser_oracle
from workloads import make_custom, make_workload


def _fwd(w, **kw):
    s = w.spec
    return laser_oracle.forward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg,
                                s.S, s.H, kw.get("gamma", w.gamma), kw.get("tau", w.tau))


# ---------------------------------------------------------------- per-segment loops == global reshaped form
@pytest.mark.parametrize("U,C,L,d,H,S,M,d_qh,lengths", [
    (1, 2, 12, 4, 1, 4, 1, 2, [12]),
    (2, 3, 24, 8, 2, 6, 2, 2, [24, 13]),
    (2, 2, 10, 8, 4, 4, 2, 1, [7, 0]),        # L not a multiple of S, an empty user
    (1, 3, 9, 6, 3, 9, 3, 2, [5]),            # one segment
    (3, 1, 16, 4, 2, 1, 1, 2, [16, 1, 9]),    # segment size 1
])
def test_brute_force_matches_vectorised(U, C, L, d, H, S, M, d_qh, lengths):
    w = make_custom(U=U, C=C, L=L, d=d, H=H, S=S, M=M, d_qh=d_qh, lengths=lengths, seed=11, emb_std="one")
    Hp, z = _fwd(w)
    Hb, zb = laser_brute.forward(w.items.tolist(), w.lengths, w.cands.tolist(), w.cand_offsets,
                                 w.Wq.tolist(), w.Wk.tolist(), w.Wv.tolist(), w.Wg.tolist(),
                                 S, H, w.gamma, w.tau)
    np.testing.assert_allclose(Hp, np.array(Hb), rtol=0, atol=1e-12)
    np.testing.assert_allclose(z, np.array(zb), rtol=0, atol=1e-12)


# ---------------------------------------------------------------- S = L: one gated target attention, closed form
def test_single_segment_closed_form():
    w = make_custom(U=1, C=4, L=20, d=8, H=1, S=20, M=3, d_qh=4, lengths=[17], seed=3, emb_std="one")
    Hp, z = _fwd(w)
    X = w.items[0].astype(np.float64)
    for c in range(4):
        t = w.cands[c].astype(np.float64)
        q = t @ w.Wq
        s0 = np.zeros(8)
        for n in range(17):
            x = X[n]
            s0 += (1.0 / (1.0 + math.exp(-float(q @ (x @ w.Wk)) / w.gamma))) * (x @ w.Wv)
        np.testing.assert_allclose(Hp[c, 0], s0, atol=1e-12)
        # softmax over a single segment is 1, so every layer adds s0 W_v^l
        z_ref = t + s0 @ (w.Wg[:, 2].astype(np.float64).sum(axis=0))
        np.testing.assert_allclose(z[c], z_ref, atol=1e-12)


# ---------------------------------------------------------------- W_q = 0: every gate is 1/2 -> sum pooling
def test_zero_query_gives_half_sum_pooling():
    w = make_custom(U=2, C=3, L=30, d=8, H=2, S=7, M=1, d_qh=2, lengths=[30, 11], seed=5)
    w.Wq[:] = 0
    Hp, _ = _fwd(w)
    for u in range(2):
        X = w.items[u].astype(np.float64).copy()
        X[w.lengths[u]:] = 0
        Xp = np.concatenate([X, np.zeros((35 - 30, 8))])
        pooled = 0.5 * Xp.reshape(5, 7, 8).sum(axis=1) @ w.Wv
        for c in range(3 * u, 3 * u + 3):
            np.testing.assert_allclose(Hp[c], pooled, atol=1e-13)


# ---------------------------------------------------------------- silence / saturation limits
def test_saturation_limits():
    w = make_custom(U=1, C=2, L=16, d=4, H=2, S=4, M=2, d_qh=2, lengths=[14], seed=9, emb_std="one")
    w.items[:] = np.abs(w.items) + 0.1
    w.cands[:] = np.abs(w.cands) + 0.1
    w.Wk[:] = np.abs(w.Wk) + 0.1
    w.Wq[:] = -(np.abs(w.Wq) + 0.1)          # every score is negative
    Hp, z = _fwd(w, gamma=1e-4)
    assert np.abs(Hp).max() < 1e-200           # gates vanish: the segment is silenced
    np.testing.assert_allclose(z, w.cands, atol=1e-12)   # attention over zero vectors adds nothing
    w.Wq[:] = -w.Wq                           # every score is large and positive: gates -> 1
    Hp, _ = _fwd(w, gamma=1e-4)
    X = w.items[0].astype(np.float64).copy()
    X[14:] = 0
    sumv = (X @ w.Wv).reshape(4, 4, 4).sum(axis=1)
    np.testing.assert_allclose(Hp[0], sumv, atol=1e-12)


# ---------------------------------------------------------------- GSTA layer == library single-query attention
def test_gsta_matches_library_attention():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(2)
    C, Lp, d, H, S = 3, 6, 8, 2, 5
    Hp = rng.standard_normal((C, Lp, d))
    T = rng.standard_normal((C, d))
    Wg = rng.standard_normal((1, 3, d, d)) / math.sqrt(d)
    ell = 22                                   # 5 non-empty segments of 6
    tau = 1.7
    z = laser_oracle.gsta_user(Hp, ell, T, Wg, S, H, tau)
    q = torch.tensor(T @ Wg[0, 0]).reshape(C, 1, H, d // H).transpose(1, 2)
    k = torch.tensor(Hp @ Wg[0, 1]).reshape(C, Lp, H, d // H).transpose(1, 2)
    v = torch.tensor(Hp @ Wg[0, 2]).reshape(C, Lp, H, d // H).transpose(1, 2)
    mask = torch.zeros(1, 1, 1, Lp, dtype=torch.bool)
    mask[..., :5] = True
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask, scale=1.0 / tau)
    z_ref = T + o.transpose(1, 2).reshape(C, d).numpy()
    np.testing.assert_allclose(z, z_ref, atol=1e-12)
    # and against scipy's softmax, one head at a time
    for c in range(C):
        o2 = np.zeros(d)
        for h in range(H):
            sl = slice(h * (d // H), (h + 1) * (d // H))
            e = (Hp[c, :5] @ Wg[0, 1])[:, sl] @ (T[c] @ Wg[0, 0])[sl] / tau
            o2[sl] = sp_softmax(e) @ (Hp[c, :5] @ Wg[0, 2])[:, sl]
        np.testing.assert_allclose(z[c], T[c] + o2, atol=1e-12)


def test_gsta_zero_query_is_mean_over_nonempty_segments():
    rng = np.random.default_rng(4)
    C, Lp, d, H, S = 2, 5, 6, 3, 4
    Hp = rng.standard_normal((C, Lp, d))
    T = rng.standard_normal((C, d))
    Wg = rng.standard_normal((2, 3, d, d))
    Wg[:, 0] = 0
    z = laser_oracle.gsta_user(Hp, 9, T, Wg, S, H, 1.0)     # ceil(9/4) = 3 non-empty segments
    ref = T + Hp[:, :3].mean(axis=1) @ (Wg[0, 2] + Wg[1, 2])
    np.testing.assert_allclose(z, ref, atol=1e-12)


def test_gsta_output_in_convex_hull_and_layers_see_same_hprime():
    rng = np.random.default_rng(6)
    C, Lp, d, H, S = 1, 4, 4, 1, 3
    Hp = rng.standard_normal((C, Lp, d))
    T = rng.standard_normal((C, d))
    Wg = rng.standard_normal((1, 3, d, d))
    z = laser_oracle.gsta_user(Hp, 12, T, Wg, S, H, 2.0)
    vals = Hp[0] @ Wg[0, 2]
    o = z[0] - T[0]
    assert np.all(o <= vals.max(axis=0) + 1e-12) and np.all(o >= vals.min(axis=0) - 1e-12)
    # two layers == applying one-layer GSTA twice with the updated target and the SAME H'
    Wg2 = rng.standard_normal((2, 3, d, d))
    z2 = laser_oracle.gsta_user(Hp, 12, T, Wg2, S, H, 2.0)
    t1 = laser_oracle.gsta_user(Hp, 12, T, Wg2[:1], S, H, 2.0)
    t2 = laser_oracle.gsta_user(Hp, 12, t1, Wg2[1:], S, H, 2.0)
    np.testing.assert_allclose(z2, t2, atol=1e-13)


# ---------------------------------------------------------------- masking, permutation, linearity, independence
def test_padding_contents_do_not_matter_and_truncation():
    w = make_custom(U=2, C=2, L=24, d=8, H=2, S=5, M=2, d_qh=2, lengths=[13, 20], seed=7)
    Hp, z = _fwd(w)
    w2 = make_custom(U=2, C=2, L=24, d=8, H=2, S=5, M=2, d_qh=2, lengths=[13, 20], seed=7)
    w2.items[0, 13:] = -3.25
    w2.items[1, 20:] = 1e3
    Hp2, z2 = _fwd(w2)
    assert np.array_equal(Hp, Hp2) and np.array_equal(z, z2)
    assert np.all(Hp[:2, 3:] == 0)             # user 0 has ceil(13/5) = 3 non-empty segments
    # truncating the sequence to the non-empty segments leaves z unchanged
    s = w.spec
    Hp3, z3 = laser_oracle.forward(w.items[:, :20], w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg,
                                   s.S, s.H, w.gamma, w.tau)
    np.testing.assert_allclose(z3, z, atol=1e-14)
    np.testing.assert_allclose(Hp3, Hp[:, :4], atol=1e-14)


def test_permutation_invariance():
    w = make_custom(U=1, C=3, L=24, d=8, H=2, S=6, M=2, d_qh=2, lengths=[24], seed=8)
    Hp, z = _fwd(w)
    rng = np.random.default_rng(0)
    items = w.items.copy()
    for i in range(4):                          # shuffle items inside each segment
        items[0, 6 * i:6 * i + 6] = items[0, 6 * i + rng.permutation(6)]
    s = w.spec
    Hp2, z2 = laser_oracle.forward(items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg,
                                   s.S, s.H, w.gamma, w.tau)
    np.testing.assert_allclose(Hp2, Hp, atol=1e-14)
    np.testing.assert_allclose(z2, z, atol=1e-14)
    perm = np.array([2, 0, 3, 1])               # shuffle whole segments
    items3 = w.items.reshape(1, 4, 6, 8)[:, perm].reshape(1, 24, 8)
    Hp3, z3 = laser_oracle.forward(items3, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg,
                                   s.S, s.H, w.gamma, w.tau)
    np.testing.assert_allclose(Hp3, Hp[:, perm], atol=1e-14)
    np.testing.assert_allclose(z3, z, atol=1e-13)


def test_value_linearity():
    w = make_custom(U=1, C=2, L=12, d=4, H=1, S=4, M=1, d_qh=2, lengths=[10], seed=1)
    Hp, _ = _fwd(w)
    w.Wv[:] = w.Wv * 4.0                        # exact in floating point
    Hp2, _ = _fwd(w)
    np.testing.assert_allclose(Hp2, 4.0 * Hp, atol=1e-14)


def test_candidates_users_and_heads_are_independent():
    w = make_custom(U=2, C=3, L=16, d=8, H=2, S=4, M=2, d_qh=2, lengths=[16, 9], seed=12)
    Hp, z = _fwd(w)
    s = w.spec
    for u in range(2):
        for c in range(3 * u, 3 * u + 3):       # one (user, candidate) at a time
            Hp1, z1 = laser_oracle.forward(w.items[u:u + 1], w.lengths[u:u + 1], w.cands[c:c + 1],
                                           np.array([0, 1]), w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H, w.gamma, w.tau)
            np.testing.assert_allclose(Hp1[0], Hp[c], atol=1e-14)
            np.testing.assert_allclose(z1[0], z[c], atol=1e-14)
    # STA with H heads == H single-head runs on the weight column slices, concatenated
    parts = []
    for h in range(2):
        Hh = laser_oracle.sta_forward(w.items, w.lengths, w.cands, w.cand_offsets,
                                      w.Wq[:, 2 * h:2 * h + 2], w.Wk[:, 2 * h:2 * h + 2], w.Wv[:, 4 * h:4 * h + 4],
                                      s.S, 1, w.gamma)
        parts.append(Hh)
    np.testing.assert_allclose(np.concatenate(parts, axis=2), Hp, atol=1e-14)


def test_default_scales():
    w = make_custom(U=1, C=1, L=8, d=8, H=2, S=4, M=1, d_qh=4, lengths=[8], seed=1)
    s = w.spec
    assert w.gamma == pytest.approx(2.0) and w.tau == pytest.approx(2.0)
    a = laser_oracle.forward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H)
    b = _fwd(w)
    assert np.array_equal(a[1], b[1])


# ---------------------------------------------------------------- the paper's printed cost numbers
def test_cost_model_reproduces_paper_numbers(repo_root):
    vals = {}
    with open(os.path.join(repo_root, "tests", "golden", "paper_cost_numbers.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v, tol = line.split()
                vals[k] = (float(v), float(tol))
    L, d, d_q, w, r, M = 1000, 128, 32, 10, 4, 2
    got = {
        "self_attention": cost_model.c_self_attention(L, d),
        "laser": cost_model.c_laser(L, d, d_q, w, r, M),
        "target_attention": cost_model.c_target_attention(L, d),
        "table_din": cost_model.c_target_attention(L, d),
        "table_laser": cost_model.c_laser(L, d, d_q, w, r, M),
        "rel_flops_w5": cost_model.c_laser(L, d, d_q, 5, r, M) / cost_model.c_laser(L, d, d_q, 10, r, M),
        "rel_flops_w20": cost_model.c_laser(L, d, d_q, 20, r, M) / cost_model.c_laser(L, d, d_q, 10, r, M),
    }
    for k, (v, tol) in vals.items():
        assert got[k] == pytest.approx(v, rel=tol), k
    # the closed total equals the sum of its stages up to the dropped lower-order terms
    parts = cost_model.c_sta(L, d, d_q, w, r) + cost_model.c_gsta(L, d, w, M)
    assert parts == pytest.approx(cost_model.c_laser(L, d, d_q, w, r, M), rel=0.01)
    # the three stage costs of the "Computational Complexity" section, counted by hand from the shapes of the products
    # at a small size: K [L x d_q] and V [L x d] from X [L x d]; one score and one weighted value per item and target;
    # two d x r d products per compressed vector
    Ls, ds, dqs, ws, rs = 12, 8, 4, 3, 2
    assert cost_model.c_proj(Ls, ds, dqs) == sum(ds for _ in range(Ls) for _ in range(dqs + ds))
    assert cost_model.c_attn(Ls, ds, dqs) == sum(dqs + ds for _ in range(Ls))
    assert cost_model.c_ffn(Ls, ds, ws, rs) == sum(ds * rs * ds + rs * ds * ds for _ in range(Ls // ws))
    # and the stage total the paper prints drops only the per-target term
    assert cost_model.c_sta(Ls, ds, dqs, ws, rs) == cost_model.c_proj(Ls, ds, dqs) + cost_model.c_ffn(Ls, ds, ws, rs)


# ---------------------------------------------------------------- the duplicate-item workload exercises the gate
def test_near_duplicate_workload_exercises_gate():
    from scipy.special import expit
    w = make_workload("cfg3", users=2)
    s = w.spec
    hi = lo = tot = 0
    for u in range(2):
        ell = int(w.lengths[u])
        X = w.items[u, :ell].astype(np.float64)
        T = w.cands[u * s.C:(u + 1) * s.C].astype(np.float64)
        cos = (X / np.linalg.norm(X, axis=1, keepdims=True)) @ (T / np.linalg.norm(T, axis=1, keepdims=True)).T
        pos, src = w.dup_pos[u]
        assert np.all(cos[pos, src] > 0.9)
        assert abs(len(pos) / ell - 0.10) < 0.01
        Q = (T @ w.Wq).reshape(s.C, s.H, s.d_qh)
        K = (X @ w.Wk).reshape(ell, s.H, s.d_qh)
        g = expit(np.einsum("chq,nhq->cnh", Q, K) / w.gamma)
        assert np.mean(g[src, pos] > 0.99) >= 0.8          # a duplicate opens the gate of its source candidate
        hi += np.sum(g > 0.8); lo += np.sum(g < 0.2); tot += g.size
    assert hi / tot >= 0.10 and lo / tot >= 0.10            # and the rest spread over the whole gate range
