"""GPU parity of the feed-forward refinement (Eq. 6) against its oracle: laser_ffn_forward on given segment vectors
(tensor-core kernel, FP32-ALU kernel) and laser_forward_ffn (STA -> Eq. 6 -> GSTA) end to end."""
import numpy as np
import pytest
import torch

import paper_2602_11562_b200 as P
from oracle import ffn_oracle, laser_oracle
from workloads import make_custom, make_ffn_weights, round_to_dtype
from _util import TOL, err_metric, to_np

pytestmark = pytest.mark.gpu

SENTINEL = 7.0      # planted in the rows of empty segments: the kernels must neither read nor write them


def _ffn_dev(fw, tdt):
    return {k: torch.from_numpy(v).to(tdt).cuda() for k, v in fw.items()}


def _oracle_ffn(Hp, w, fw):
    return ffn_oracle.ffn_forward(Hp, w.lengths, w.cand_offsets, w.spec.S, fw["W1"], fw["b1"], fw["W2"], fw["b2"],
                                  fw["ln_g"], fw["ln_b"])


CASES = [
    # tensor-core kernel (bf16, d % 16 == 0, hidden % 128 == 0)
    dict(U=3, C=40, L=256, d=128, S=16, r=4, dtype="bf16", lengths=[256, 100, 0]),      # 4 chunks; several tile pairs, ragged tail
    dict(U=2, C=7, L=96, d=64, S=24, r=4, dtype="bf16", lengths=[96, 1]),               # 2 chunks; less than one tile
    dict(U=4, C=33, L=128, d=96, S=8, r=4, dtype="bf16", lengths=[128, 9, 64, 127]),    # 3 chunks, 12 pieces per row
    dict(U=2, C=70, L=64, d=32, S=4, r=4, dtype="bf16", lengths=[64, 30]),              # 1 chunk
    dict(U=5, C=130, L=160, d=128, S=10, r=2, dtype="bf16", lengths=[160, 0, 155, 10, 77]),   # r = 2; > 148 pairs? no: many rows
    dict(U=1, C=1, L=16, d=16, S=16, r=8, dtype="bf16", lengths=[5]),                   # a single row
    # FP32-ALU kernel
    dict(U=3, C=5, L=70, d=24, S=16, r=4, dtype="f32", lengths=[70, 33, 0]),
    dict(U=2, C=9, L=40, d=64, S=8, r=3, dtype="f32", lengths=[40, 17]),
    dict(U=2, C=6, L=48, d=40, S=16, r=3, dtype="bf16", lengths=[48, 20]),              # bf16, hidden = 120: not a chunk multiple
]


@pytest.mark.parametrize("case", range(len(CASES)))
def test_ffn_matches_oracle(case):
    kw = dict(CASES[case])
    r, dtype = kw.pop("r"), kw["dtype"]
    H = 1 if kw["d"] % 32 else 2
    w = make_custom(H=H, M=1, seed=700 + case, **kw)
    s = w.spec
    if case == 0:
        w.cand_offsets = np.array([0, 50, 50, 120], dtype=np.int32)   # uneven; user 1 has no candidates
        w.lengths = np.array([256, 100, 77], dtype=np.int32)
    fw = make_ffn_weights(s.d, r, dtype, seed=case)
    rng = np.random.default_rng(case)
    N, Lp = int(w.cand_offsets[-1]), s.n_seg
    Hp = round_to_dtype((0.7 * rng.standard_normal((N, Lp, s.d))).astype(np.float32), dtype)
    live = np.zeros((N, Lp), dtype=bool)
    for u in range(s.U):
        n = -(-int(w.lengths[u]) // s.S)
        live[int(w.cand_offsets[u]):int(w.cand_offsets[u + 1]), :n] = True
    Hp[~live] = SENTINEL
    ref = _oracle_ffn(np.where(live[..., None], Hp, 0.0), w, fw)
    b = P.DeviceBatch.from_numpy(items=w.items, lengths=w.lengths, cands=w.cands[:N], cand_offsets=w.cand_offsets,
                                 Wq=w.Wq, Wk=w.Wk, Wv=w.Wv, Wg=w.Wg, S=s.S, H=s.H, M=s.M, dtype=dtype)
    tdt = b.items.dtype
    hid = r * s.d
    ws = torch.empty(P.laser_ffn_workspace_bytes(b.cfg, hid), dtype=torch.uint8, device="cuda")
    Hd = torch.from_numpy(Hp).to(tdt).cuda()
    P.laser_ffn_forward(b.cfg, _ffn_dev(fw, tdt), Hd, b.lengths, b.cand_offsets, workspace=ws)
    assert P.laser_check_status(ws) == 0
    got = to_np(Hd)
    assert np.all(got[~live] == SENTINEL)
    e = err_metric(got[live], ref[live])
    assert e <= TOL[dtype], f"case {case}: err {e}"
    names = [n for n, _ in _profile(b, fw, Hp, tdt, hid)]
    want_tc = dtype == "bf16" and s.d % 16 == 0 and hid % 128 == 0
    assert ("ffn_tc" in names) == want_tc, names


def _profile(b, fw, Hp, tdt, hid):
    ws = torch.empty(P.laser_ffn_workspace_bytes(b.cfg, hid), dtype=torch.uint8, device="cuda")
    P.laser_profile_enable(True)
    try:
        P.laser_ffn_forward(b.cfg, _ffn_dev(fw, tdt), torch.from_numpy(Hp).to(tdt).cuda(), b.lengths, b.cand_offsets,
                            workspace=ws)
        return P.laser_profile_read()
    finally:
        P.laser_profile_enable(False)


def test_ffn_simt_path_on_a_tensor_shape_agrees_too():
    w = make_custom(U=2, C=20, L=64, d=64, H=2, S=16, M=1, dtype="bf16", seed=733, lengths=[64, 40])
    s = w.spec
    fw = make_ffn_weights(s.d, 4, "bf16", seed=33)
    rng = np.random.default_rng(33)
    Hp = round_to_dtype(rng.standard_normal((w.N, s.n_seg, s.d)).astype(np.float32), "bf16")
    Hp[20:, 3:] = 0.0                                                  # user 1: 3 non-empty segments
    ref = _oracle_ffn(Hp, w, fw)
    b = P.DeviceBatch.from_workload(w, path=P.PATH_SIMT)
    Hd = torch.from_numpy(Hp).to(torch.bfloat16).cuda()
    P.laser_ffn_forward(b.cfg, _ffn_dev(fw, torch.bfloat16), Hd, b.lengths, b.cand_offsets)
    assert err_metric(to_np(Hd), ref) <= TOL["bf16"]


@pytest.mark.parametrize("dtype,path", [("bf16", P.PATH_AUTO), ("f32", P.PATH_AUTO), ("bf16", P.PATH_STREAM)])
def test_forward_with_ffn_matches_the_composed_oracle(dtype, path):
    C = 1 if path == P.PATH_STREAM else 140
    U = 40 if path == P.PATH_STREAM else 3
    lengths = None if path == P.PATH_STREAM else [384, 130, 0]
    w = make_custom(U=U, C=C, L=384, d=64, H=2, S=32, M=2, dtype=dtype, seed=741, lengths=lengths)
    s = w.spec
    fw = make_ffn_weights(s.d, 4, dtype, seed=41)
    Hp0 = laser_oracle.sta_forward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, s.S, s.H, w.gamma)
    Hp1 = _oracle_ffn(Hp0, w, fw)
    z_ref = laser_oracle.gsta_forward(Hp1, w.lengths, w.cand_offsets, w.cands, w.Wg, s.S, s.H, w.tau)
    b = P.DeviceBatch.from_workload(w, path=path)
    tdt = b.items.dtype
    ws = torch.empty(P.laser_ffn_workspace_bytes(b.cfg, 4 * s.d), dtype=torch.uint8, device="cuda")
    Hp, z = P.laser_forward_ffn(b.cfg, *b.args(), b.Wg, _ffn_dev(fw, tdt), workspace=ws, want_hprime=True)
    assert P.laser_check_status(ws) == 0
    assert err_metric(to_np(Hp), Hp1) <= TOL[dtype]
    assert err_metric(to_np(z), z_ref) <= TOL[dtype]
    # without an H' buffer the same z comes out
    z2 = P.laser_forward_ffn(b.cfg, *b.args(), b.Wg, _ffn_dev(fw, tdt), workspace=ws)
    assert torch.equal(z2, z)


def test_ffn_rejects_bad_arguments():
    w = make_custom(U=1, C=2, L=32, d=32, H=2, S=16, M=1, dtype="bf16", seed=750)
    b = P.DeviceBatch.from_workload(w)
    fw = _ffn_dev(make_ffn_weights(32, 4, "bf16"), torch.bfloat16)
    Hd = torch.zeros((w.N, 2, 32), dtype=torch.bfloat16, device="cuda")
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(P.LaserError) as ei:
        P.laser_ffn_forward(b.cfg, fw, Hd, b.lengths, b.cand_offsets, workspace=small)
    assert ei.value.status == -3
    assert P.laser_ffn_workspace_bytes(b.cfg, 0) == 0


def test_ffn_many_users_and_no_rows_at_all():
    # More users than the set-up scan has threads (several users per thread), a third of them empty; then a batch in
    # which no segment holds an item (nothing to do, nothing touched).
    rng = np.random.default_rng(760)
    U, d, S, L = 2500, 32, 16, 64
    lengths = rng.integers(0, L + 1, size=U)
    lengths[rng.random(U) < 0.33] = 0
    w = make_custom(U=U, C=1, L=L, d=d, H=2, S=S, M=1, dtype="bf16", seed=760, lengths=lengths.tolist())
    fw = make_ffn_weights(d, 4, "bf16", seed=60)
    Lp = w.spec.n_seg
    Hp = round_to_dtype(rng.standard_normal((U, Lp, d)).astype(np.float32), "bf16")
    live = np.arange(Lp)[None, :] < (-(-lengths // S))[:, None]
    Hp[~live] = SENTINEL
    ref = _oracle_ffn(np.where(live[..., None], Hp, 0.0), w, fw)
    b = P.DeviceBatch.from_workload(w)
    ws = torch.empty(P.laser_ffn_workspace_bytes(b.cfg, 4 * d), dtype=torch.uint8, device="cuda")
    Hd = torch.from_numpy(Hp).to(torch.bfloat16).cuda()
    P.laser_ffn_forward(b.cfg, _ffn_dev(fw, torch.bfloat16), Hd, b.lengths, b.cand_offsets, workspace=ws)
    assert P.laser_check_status(ws) == 0
    got = to_np(Hd)
    assert np.all(got[~live] == SENTINEL)
    assert err_metric(got[live], ref[live]) <= TOL["bf16"]

    w0 = make_custom(U=3, C=4, L=L, d=d, H=2, S=S, M=1, dtype="bf16", seed=761, lengths=[0, 0, 0])
    b0 = P.DeviceBatch.from_workload(w0)
    H0 = torch.full((12, Lp, d), SENTINEL, dtype=torch.bfloat16, device="cuda")
    ws0 = torch.empty(P.laser_ffn_workspace_bytes(b0.cfg, 4 * d), dtype=torch.uint8, device="cuda")
    P.laser_ffn_forward(b0.cfg, _ffn_dev(fw, torch.bfloat16), H0, b0.lengths, b0.cand_offsets, workspace=ws0)
    assert P.laser_check_status(ws0) == 0
    assert bool((H0 == SENTINEL).all())
