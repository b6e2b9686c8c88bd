"""Pins of the backward oracle (oracle/backward_oracle.py) against things other than itself: central finite differences
through the forward oracle, torch.autograd through an independent per-segment restatement of the forward, and cases
whose gradient is known in closed form."""
import numpy as np
import pytest
import torch

from oracle import backward_oracle, laser_oracle
from workloads import make_custom

CASES = [
    dict(U=2, C=3, L=20, d=8, H=2, S=6, M=2, lengths=[20, 7], d_qh=4),       # ragged, a short last segment
    dict(U=3, C=2, L=12, d=6, H=1, S=4, M=1, lengths=[12, 0, 5], d_qh=3),    # an empty user, one head
    dict(U=1, C=4, L=9, d=8, H=4, S=3, M=3, lengths=[8], d_qh=2),            # three layers, four heads
]


def _case(i):
    kw = dict(CASES[i])
    w = make_custom(seed=700 + i, dtype="f32", emb_std="one", **kw)
    rng = np.random.default_rng(70 + i)
    dz = rng.standard_normal((w.N, w.spec.d))
    return w, dz


def _loss(w, dz, **over):
    a = dict(items=w.items, cands=w.cands, Wq=w.Wq, Wk=w.Wk, Wv=w.Wv, Wg=w.Wg)
    a.update(over)
    s = w.spec
    _, z = laser_oracle.forward(a["items"], w.lengths, a["cands"], w.cand_offsets, a["Wq"], a["Wk"], a["Wv"], a["Wg"], s.S,
                                s.H, w.gamma, w.tau, return_hprime=False)
    return float((z * dz).sum())


def _grads(w, dz):
    s = w.spec
    return backward_oracle.backward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H, dz,
                                    w.gamma, w.tau)


@pytest.mark.parametrize("case", range(len(CASES)))
def test_finite_differences_through_the_forward_oracle(case):
    w, dz = _case(case)
    g = _grads(w, dz)
    rng = np.random.default_rng(5)
    names = {"items": "d_items", "cands": "d_cands", "Wq": "dWq", "Wk": "dWk", "Wv": "dWv", "Wg": "dWg"}
    eps = 1e-6
    for inp, out in names.items():
        base = np.asarray(getattr(w, inp), dtype=np.float64)
        for _ in range(12):
            idx = tuple(int(rng.integers(0, n)) for n in base.shape)
            hi, lo = base.copy(), base.copy()
            hi[idx] += eps
            lo[idx] -= eps
            fd = (_loss(w, dz, **{inp: hi}) - _loss(w, dz, **{inp: lo})) / (2 * eps)
            assert abs(fd - g[out][idx]) <= 1e-6 * max(1.0, abs(fd)), (inp, idx, fd, g[out][idx])


def _torch_forward(items, lengths, cands, offs, Wq, Wk, Wv, Wg, S, H, gamma, tau):
    """The forward written segment by segment and head by head with scalar-indexed torch ops (Eq. 4-5, Eq. 7)."""
    U, L, d = items.shape
    dqh, dvh = Wq.shape[1] // H, d // H
    zs = []
    for u in range(U):
        for c in range(int(offs[u]), int(offs[u + 1])):
            t = cands[c]
            segs = []
            for i in range(0, int(lengths[u]), S):
                n1 = min(i + S, int(lengths[u]))
                parts = []
                for h in range(H):
                    q = t @ Wq[:, h * dqh:(h + 1) * dqh]
                    k = items[u, i:n1] @ Wk[:, h * dqh:(h + 1) * dqh]
                    v = items[u, i:n1] @ Wv[:, h * dvh:(h + 1) * dvh]
                    parts.append((torch.sigmoid(k @ q / gamma)[:, None] * v).sum(0))
                segs.append(torch.cat(parts))
            if segs:
                Hs = torch.stack(segs)
                for l in range(Wg.shape[0]):
                    outs = []
                    for h in range(H):
                        sl = slice(h * dvh, (h + 1) * dvh)
                        a = torch.softmax((Hs @ Wg[l, 1][:, sl]) @ (t @ Wg[l, 0][:, sl]) / tau, dim=0)
                        outs.append(a @ (Hs @ Wg[l, 2][:, sl]))
                    t = t + torch.cat(outs)
            zs.append(t)
    return torch.stack(zs)


@pytest.mark.parametrize("case", range(len(CASES)))
def test_autograd_through_a_per_segment_restatement(case):
    w, dz = _case(case)
    s = w.spec
    g = _grads(w, dz)
    tens = {k: torch.tensor(np.asarray(getattr(w, k), dtype=np.float64), requires_grad=True)
            for k in ("items", "cands", "Wq", "Wk", "Wv", "Wg")}
    z = _torch_forward(tens["items"], w.lengths, tens["cands"], w.cand_offsets, tens["Wq"], tens["Wk"], tens["Wv"],
                       tens["Wg"], s.S, s.H, w.gamma, w.tau)
    (z * torch.tensor(dz)).sum().backward()
    for k, out in (("items", "d_items"), ("cands", "d_cands"), ("Wq", "dWq"), ("Wk", "dWk"), ("Wv", "dWv"), ("Wg", "dWg")):
        ref = tens[k].grad.numpy()
        assert np.max(np.abs(ref - g[out])) <= 1e-10 * max(1.0, np.max(np.abs(ref))), k


def test_closed_forms_and_invariants():
    w, dz = _case(0)
    s = w.spec
    g = _grads(w, dz)
    # padding rows receive no gradient, and their contents do not matter
    for u in range(s.U):
        assert np.all(g["d_items"][u, int(w.lengths[u]):] == 0.0)
    items2 = np.array(w.items, dtype=np.float64)
    items2[1, int(w.lengths[1]):] = 123.0
    g2 = backward_oracle.backward(items2, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H, dz,
                                  w.gamma, w.tau)
    for k in g:
        assert np.allclose(g[k], g2[k], rtol=0, atol=1e-12), k
    # linear in dz
    g3 = _grads(w, -2.5 * dz)
    for k in g:
        assert np.allclose(g3[k], -2.5 * g[k], rtol=1e-12, atol=1e-12), k
    # without GSTA layers z = t: dz goes straight to the candidates and nowhere else
    g0 = backward_oracle.backward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg[:0], s.S, s.H, dz,
                                  w.gamma, w.tau)
    assert np.array_equal(g0["d_cands"], dz)
    assert all(not np.any(g0[k]) for k in ("d_items", "dWq", "dWk", "dWv"))
    # W_v^l = 0 in every layer: o_l = 0, z = t, same conclusion for everything but dW_v^l
    Wg0 = np.array(w.Wg, dtype=np.float64)
    Wg0[:, 2] = 0.0
    gz = backward_oracle.backward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, Wg0, s.S, s.H, dz,
                                  w.gamma, w.tau)
    assert np.allclose(gz["d_cands"], dz, atol=1e-14) and not np.any(gz["d_items"]) and not np.any(gz["dWg"][:, :2])
    assert np.any(gz["dWg"][:, 2])
    # a user restricted run equals the rows of the full run
    gu = backward_oracle.backward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H, dz,
                                  w.gamma, w.tau, users=[1])
    assert np.allclose(gu["d_items"][1], g["d_items"][1], atol=1e-14) and not np.any(gu["d_items"][0])
