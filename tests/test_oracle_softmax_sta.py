"""Pins for the oracle of the softmax-aggregation STA variant."""
import math

import numpy as np
from scipy.special import softmax

from oracle import softmax_sta_oracle as so


def _case(seed, L=11, d=6, dqk=4, C=3):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((L, d)), rng.standard_normal((C, d)), rng.standard_normal((d, dqk)),
            rng.standard_normal((d, dqk)), rng.standard_normal((d, d)))


def test_matches_scalar_loops():
    X, T, Wq, Wk, Wv = _case(1)
    S, H, gamma, ell = 4, 2, 1.7, 9
    got = so.sta_softmax_user(X, ell, T, Wq, Wk, Wv, S, H, gamma)
    L, d = X.shape
    dqh, dvh = Wq.shape[1] // H, d // H
    for c in range(T.shape[0]):
        q = [sum(T[c, k] * Wq[k, j] for k in range(d)) for j in range(Wq.shape[1])]
        for i in range(-(-L // S)):
            items = [n for n in range(i * S, min((i + 1) * S, L)) if n < ell]
            for h in range(H):
                want = [0.0] * dvh
                if items:
                    sc = []
                    for n in items:
                        kk = [sum(X[n, k] * Wk[k, h * dqh + a] for k in range(d)) for a in range(dqh)]
                        sc.append(sum(q[h * dqh + a] * kk[a] for a in range(dqh)) / gamma)
                    mx = max(sc)
                    w = [math.exp(x - mx) for x in sc]
                    z = sum(w)
                    for wn, n in zip(w, items):
                        for e in range(dvh):
                            want[e] += wn / z * sum(X[n, k] * Wv[k, h * dvh + e] for k in range(d))
                np.testing.assert_allclose(got[c, i, h * dvh:(h + 1) * dvh], want, atol=1e-12)


def test_matches_scipy_softmax_on_a_full_segment():
    X, T, Wq, Wk, Wv = _case(2, L=8)
    H, gamma = 1, 0.9
    got = so.sta_softmax_user(X, 8, T, Wq, Wk, Wv, 8, H, gamma)[:, 0]
    a = softmax((T @ Wq) @ (X @ Wk).T / gamma, axis=1)
    np.testing.assert_allclose(got, a @ (X @ Wv), atol=1e-12)


def test_zero_query_weights_give_mean_pooling_and_one_item_segments_give_the_value():
    X, T, Wq, Wk, Wv = _case(3, L=10)
    got = so.sta_softmax_user(X, 7, T, np.zeros_like(Wq), Wk, Wv, 4, 2, 1.0)
    V = X @ Wv
    np.testing.assert_allclose(got[:, 0], np.broadcast_to(V[0:4].mean(axis=0), got[:, 0].shape), atol=1e-12)
    np.testing.assert_allclose(got[:, 1], np.broadcast_to(V[4:7].mean(axis=0), got[:, 1].shape), atol=1e-12)   # 3 valid items
    assert not got[:, 2].any()                                                                                 # empty segment
    one = so.sta_softmax_user(X, 10, T, Wq, Wk, Wv, 1, 2, 1.0)
    np.testing.assert_allclose(one, np.broadcast_to(V[None], one.shape), atol=1e-12)


def test_small_gamma_picks_the_best_item_per_head():
    X, T, Wq, Wk, Wv = _case(4, L=6)
    H = 2
    got = so.sta_softmax_user(X, 6, T, Wq, Wk, Wv, 6, H, 1e-4)[:, 0]
    Q, K, V = T @ Wq, X @ Wk, X @ Wv
    dqh, dvh = Wq.shape[1] // H, X.shape[1] // H
    for c in range(T.shape[0]):
        for h in range(H):
            n = int(np.argmax(K[:, h * dqh:(h + 1) * dqh] @ Q[c, h * dqh:(h + 1) * dqh]))
            np.testing.assert_allclose(got[c, h * dvh:(h + 1) * dvh], V[n, h * dvh:(h + 1) * dvh], atol=1e-9)


def test_weights_are_convex_and_padding_is_irrelevant():
    X, T, Wq, Wk, Wv = _case(5, L=12)
    ell, S, H = 10, 5, 2
    got = so.sta_softmax_user(X, ell, T, Wq, Wk, Wv, S, H, 1.3)
    V = X @ Wv
    for i, (n0, n1) in enumerate([(0, 5), (5, 10)]):
        assert np.all(got[:, i] <= V[n0:n1].max(axis=0) + 1e-12) and np.all(got[:, i] >= V[n0:n1].min(axis=0) - 1e-12)
    assert not got[:, 2].any()
    X2 = X.copy()
    X2[ell:] = 1e3
    np.testing.assert_array_equal(so.sta_softmax_user(X2, ell, T, Wq, Wk, Wv, S, H, 1.3), got)
    # a constant added to every key of a head (here: a key bias along q) cannot change softmax weights; the sigmoid gate
    # would change: check the invariance through an equivalent construction, scaling all scores' offsets via T = 0
    zero_t = so.sta_softmax_user(X, ell, np.zeros_like(T), Wq, Wk, Wv, S, H, 1.3)
    np.testing.assert_allclose(zero_t[:, 0], np.broadcast_to(V[0:5].mean(axis=0), zero_t[:, 0].shape), atol=1e-12)


def test_batched_wrapper_places_users():
    rng = np.random.default_rng(6)
    items = rng.standard_normal((2, 9, 4))
    cands = rng.standard_normal((5, 4))
    Wq, Wk, Wv = rng.standard_normal((4, 2)), rng.standard_normal((4, 2)), rng.standard_normal((4, 4))
    offs = np.array([0, 2, 5])
    out = so.sta_softmax_forward(items, [9, 4], cands, offs, Wq, Wk, Wv, 3, 1, 1.0)
    np.testing.assert_array_equal(out[:2], so.sta_softmax_user(items[0], 9, cands[:2], Wq, Wk, Wv, 3, 1, 1.0))
    np.testing.assert_array_equal(out[2:], so.sta_softmax_user(items[1], 4, cands[2:], Wq, Wk, Wv, 3, 1, 1.0))
