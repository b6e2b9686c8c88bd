"""GPU parity on seeded random shapes: every path that accepts the shape, against the oracle.  The shapes are drawn to
hit what hand-picked cases may miss: odd segment sizes, lengths of 0 and 1, segment counts around the 16- and 32-vector
chunk sizes, candidate counts around the 128-candidate tile, one to eight heads, zero to three GSTA layers."""
import numpy as np
import pytest
import torch

import paper_2602_11562_b200 as P
from workloads import make_custom

from _util import TOL, err_metric, oracle_forward, to_np

pytestmark = pytest.mark.gpu

PATHS = {"simt": P.PATH_SIMT, "tensor": P.PATH_TENSOR, "stream": P.PATH_STREAM, "auto": P.PATH_AUTO}


def _draw(i):
    rng = np.random.default_rng(9000 + i)
    d = int(rng.choice([16, 32, 48, 64, 96, 128]))
    heads = [h for h in (1, 2, 3, 4, 6, 8) if d % (16 * h) == 0]
    H = int(rng.choice(heads))
    U = int(rng.integers(1, 5))
    one_cand = bool(rng.random() < 0.25)
    C = 1 if one_cand else int(rng.choice([1, 2, 7, 33, 127, 128, 129, 200]))
    L = int(rng.integers(1, 400))
    S = int(rng.choice([1, 2, 7, 10, 16, 17, 31, 32, 33, 50, 64, 100, 128, 129, max(1, L)]))
    S = max(1, min(S, L))
    M = int(rng.integers(0, 4))
    kinds = rng.integers(0, 4, size=U)
    lengths = [0 if k == 0 else 1 if k == 1 else L if k == 2 else int(rng.integers(1, L + 1)) for k in kinds]
    return dict(U=U, C=C, L=L, d=d, H=H, S=S, M=M, d_qh=16, lengths=lengths)


@pytest.mark.parametrize("i", range(24))
def test_random_shape_every_path(i):
    kw = _draw(i)
    ran = []
    for dtype in ("bf16", "f32"):
        w = make_custom(dtype=dtype, seed=9100 + i, emb_std="inv_sqrt_d", **kw)
        Hp_ref, z_ref = oracle_forward(w)
        for name, path in PATHS.items():
            b = P.DeviceBatch.from_workload(w, path=path)
            need = P.laser_workspace_bytes(b.cfg)
            if need == 0:                                   # this path does not take the shape (or the dtype)
                continue
            ws = torch.empty(need, dtype=torch.uint8, device="cuda")
            Hp, z = P.laser_forward(b.cfg, *b.args(), b.Wg, workspace=ws, want_hprime=True)
            assert P.laser_check_status(ws) == 0, (kw, dtype, name)
            e_hp, e_z = err_metric(to_np(Hp), Hp_ref), err_metric(to_np(z), z_ref)
            assert e_hp <= TOL[dtype] and e_z <= TOL[dtype], (kw, dtype, name, e_hp, e_z)
            ran.append((dtype, name))
    assert ("f32", "simt") in ran and ("bf16", "auto") in ran, (kw, ran)


@pytest.mark.parametrize("i", range(12))
def test_random_shape_softmax_variant_and_backward(i):
    from oracle import backward_oracle, softmax_sta_oracle
    kw = _draw(100 + i)
    kw["L"] = min(kw["L"], 160)                             # (the float64 backward oracle is the slow side here)
    kw["S"] = min(kw["S"], kw["L"])
    kw["lengths"] = [min(x, kw["L"]) for x in kw["lengths"]]
    for dtype in ("bf16", "f32"):
        w = make_custom(dtype=dtype, seed=9300 + i, emb_std="inv_sqrt_d", **kw)
        s = w.spec
        b = P.DeviceBatch.from_workload(w)
        # the softmax-aggregation variant, whichever version takes the shape
        ref = softmax_sta_oracle.sta_softmax_forward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, s.S,
                                                     s.H, w.gamma)
        ws = torch.empty(P.laser_sta_softmax_workspace_bytes(b.cfg), dtype=torch.uint8, device="cuda")
        Hs = P.laser_sta_softmax_forward(b.cfg, *b.args(), workspace=ws)
        assert P.laser_check_status(ws) == 0
        assert err_metric(to_np(Hs), ref) <= TOL[dtype], (kw, dtype)
        # the backward pass: the automatic choice (tensor cores for bf16 batches of supported head widths: the bf16 bar of
        # tests/test_gpu_backward.py) and, for bf16, the FP32-ALU kernels on request (the fp32 bar)
        dz = np.random.default_rng(9400 + i).standard_normal((w.N, s.d)).astype(np.float32)
        want = backward_oracle.backward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H,
                                        dz.astype(np.float64), w.gamma, w.tau)
        for path, bar in ((P.PATH_AUTO, 2e-2 if dtype == "bf16" else 1e-4),) + (((P.PATH_SIMT, 1e-4),) if dtype == "bf16" else ()):
            bb = P.DeviceBatch.from_workload(w, path=path)
            ws = torch.empty(P.laser_backward_workspace_bytes(bb.cfg), dtype=torch.uint8, device="cuda")
            got = P.laser_backward(bb.cfg, *bb.args(), bb.Wg, torch.from_numpy(dz).cuda(), workspace=ws)
            assert P.laser_check_status(ws) == 0
            for k, r in want.items():
                if r.size == 0:
                    continue
                g = got[k].cpu().numpy().astype(np.float64)
                scale = max(float(np.max(np.abs(r))), 1e-30)
                assert np.max(np.abs(g - r)) <= bar * scale, (kw, dtype, path, k, float(np.max(np.abs(g - r))), scale)
