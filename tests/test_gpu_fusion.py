"""GPU parity of laser_fusion_forward against the fusion oracle.  Max pooling and copies are exact, so the comparison
is bit for bit on inputs that are exactly representable in the I/O dtype."""
import numpy as np
import pytest
import torch

import paper_2602_11562_b200 as P
from oracle import fusion_oracle
from workloads import make_custom, round_to_dtype

pytestmark = pytest.mark.gpu

CASES = [
    # U, C, L, d, S, dtype, lengths, num_recent
    dict(U=3, C=5, L=70, d=32, S=16, dtype="f32", lengths=[70, 33, 0], r=2),          # an empty user, fp32
    dict(U=2, C=37, L=96, d=64, S=24, dtype="bf16", lengths=[96, 1], r=3),            # one-segment user, r > its segments
    dict(U=2, C=9, L=640, d=128, S=10, dtype="bf16", lengths=[640, 333], r=4),        # 64 segments, 16 pieces per row
    dict(U=4, C=3, L=100, d=96, S=25, dtype="bf16", lengths=[100, 26, 50, 99], r=0),  # 12 pieces per row, no recent slots
    dict(U=1, C=130, L=64, d=16, S=8, dtype="bf16", lengths=[60], r=8),               # 2 pieces per row, r = L'
    dict(U=2, C=4, L=48, d=256, S=16, dtype="f32", lengths=[48, 17], r=1),            # 64 pieces per row (> one warp)
]


@pytest.mark.parametrize("case", range(len(CASES)))
def test_fusion_matches_oracle_bit_for_bit(case):
    kw = dict(CASES[case])
    r, dtype = kw.pop("r"), kw["dtype"]
    H = 1 if kw["d"] % 32 else 2
    w = make_custom(H=H, M=1, seed=500 + case, **kw)
    s = w.spec
    rng = np.random.default_rng(case)
    N, Lp = w.N, s.n_seg
    Hp = round_to_dtype((rng.standard_normal((N, Lp, s.d)) - 0.5).astype(np.float32), dtype)
    z = round_to_dtype(rng.standard_normal((N, s.d)).astype(np.float32), dtype)
    if case == 0:
        w.cand_offsets = np.array([0, 7, 7, 15], dtype=np.int32)       # uneven, a user without candidates
    for u in range(s.U):                                               # rows of empty segments must never be read
        n = -(-int(w.lengths[u]) // s.S)
        Hp[int(w.cand_offsets[u]):int(w.cand_offsets[u + 1]), n:, :] = np.float32("nan")
    ref = fusion_oracle.fusion_forward(np.nan_to_num(Hp), z, w.lengths, w.cand_offsets, s.S, r)
    b = P.DeviceBatch.from_workload(w, path=P.PATH_SIMT)
    tdt = b.items.dtype
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    out = P.laser_fusion_forward(b.cfg, torch.from_numpy(Hp).to(tdt).cuda(), torch.from_numpy(z).to(tdt).cuda(),
                                 b.lengths, b.cand_offsets, r, workspace=ws)
    assert P.laser_check_status(ws) == 0
    got = out.float().cpu().numpy().astype(np.float64)
    assert got.shape == ref.shape
    np.testing.assert_array_equal(got, ref)


def test_fusion_after_forward_on_a_tensor_path_batch():
    """End to end: H' and z from laser_forward, fused on the GPU, against the oracle applied to the same H' and z."""
    w = make_custom(U=2, C=150, L=512, d=64, H=4, S=64, M=2, dtype="bf16", seed=61, lengths=[512, 201])
    b = P.DeviceBatch.from_workload(w)
    wsf = torch.empty(P.laser_workspace_bytes(b.cfg), dtype=torch.uint8, device="cuda")
    Hp, z = P.laser_forward(b.cfg, *b.args(), b.Wg, workspace=wsf, want_hprime=True)
    out = P.laser_fusion_forward(b.cfg, Hp, z, b.lengths, b.cand_offsets, 2)
    ref = fusion_oracle.fusion_forward(Hp.float().cpu().numpy(), z.float().cpu().numpy(), w.lengths, w.cand_offsets,
                                       w.spec.S, 2)
    np.testing.assert_array_equal(out.float().cpu().numpy().astype(np.float64), ref)
