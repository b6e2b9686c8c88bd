"""laser_forward_packed (items stored without padding) against laser_forward on the padded copy of the same batch
(same kernels, same arithmetic: bit for bit) and against the oracle."""
import numpy as np
import pytest
import torch

import paper_2602_11562_b200 as P
from workloads import make_custom
from _util import TOL, err_metric, oracle_forward, to_np

pytestmark = pytest.mark.gpu

CASES = [
    # path, workload
    ("simt", dict(U=3, C=5, L=70, d=32, H=2, S=16, M=1, dtype="f32", lengths=[70, 33, 0])),
    ("tensor", dict(U=3, C=130, L=700, d=128, H=4, S=128, M=2, dtype="bf16", lengths=[700, 129, 0])),
    ("tensor", dict(U=4, C=40, L=1000, d=64, H=2, S=100, M=2, dtype="bf16", lengths=[1000, 250, 3, 999])),
    ("stream", dict(U=37, C=1, L=300, d=64, H=2, S=64, M=1, dtype="bf16", lengths=None)),
]
PATHS = {"simt": P.PATH_SIMT, "tensor": P.PATH_TENSOR, "stream": P.PATH_STREAM}


@pytest.mark.parametrize("case", range(len(CASES)))
def test_packed_layout_matches_padded_layout_and_oracle(case):
    path, kw = CASES[case]
    w = make_custom(seed=950 + case, **kw)
    s = w.spec
    b = P.DeviceBatch.from_workload(w, path=PATHS[path])
    ws = torch.empty(P.laser_workspace_bytes(b.cfg), dtype=torch.uint8, device="cuda")
    Hp_pad, z_pad = P.laser_forward(b.cfg, *b.args(), b.Wg, workspace=ws, want_hprime=True)
    assert P.laser_check_status(ws) == 0
    lens = w.lengths.astype(np.int64)
    offs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    packed = np.concatenate([w.items[u, :lens[u]] for u in range(s.U)] + [np.zeros((0, s.d), np.float32)], axis=0)
    tdt = b.items.dtype
    items_p = torch.from_numpy(np.ascontiguousarray(packed)).to(tdt).cuda()
    if items_p.numel() == 0:
        items_p = torch.zeros((1, s.d), dtype=tdt, device="cuda")
    offs_d = torch.from_numpy(offs).cuda()
    Hp, z = P.laser_forward_packed(b.cfg, items_p, offs_d, b.lengths, b.cands, b.cand_offsets, b.Wq, b.Wk, b.Wv, b.Wg,
                                   workspace=ws, want_hprime=True)
    assert P.laser_check_status(ws) == 0
    assert torch.equal(Hp, Hp_pad) and torch.equal(z, z_pad)
    Hp_ref, z_ref = oracle_forward(w)
    assert err_metric(to_np(Hp), Hp_ref) <= TOL[s.dtype]
    assert err_metric(to_np(z), z_ref) <= TOL[s.dtype]


def test_packed_layout_reports_rows_outside_the_array():
    w = make_custom(U=2, C=130, L=256, d=64, H=2, S=64, M=1, dtype="bf16", seed=960, lengths=[256, 100])
    b = P.DeviceBatch.from_workload(w, path=P.PATH_TENSOR)
    ws = torch.empty(P.laser_workspace_bytes(b.cfg), dtype=torch.uint8, device="cuda")
    items_p = torch.zeros((356, 64), dtype=torch.bfloat16, device="cuda")
    bad_offs = torch.tensor([0, 300, 356], dtype=torch.int32, device="cuda")      # user 1's 100 rows would end at 400 > 356
    z = P.laser_forward_packed(b.cfg, items_p, bad_offs, b.lengths, b.cands, b.cand_offsets, b.Wq, b.Wk, b.Wv, b.Wg,
                               workspace=ws)
    assert P.laser_check_status(ws) == -6
    assert torch.isfinite(z.float()).all()
