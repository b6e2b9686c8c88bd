"""laser_sta_forward_static: the workspace-free STA entry point for callers that cannot allocate device memory
(its scratch is a fixed array inside the library).  Collected last on purpose, so that a run stopping at the first
failure has already been through every other test."""
import pytest
import torch

import paper_2602_11562_b200 as P
from oracle import laser_oracle
from workloads import make_custom

from _util import TOL, err_metric, to_np

pytestmark = pytest.mark.gpu


def _both(w):
    """Same inputs through the existing entry point (caller-allocated workspace) and the workspace-free one."""
    b = P.DeviceBatch.from_workload(w, path=P.PATH_SIMT)
    ref = P.laser_sta_forward(b.cfg, *b.args())
    out = torch.full_like(ref, float("nan"))          # caller-owned output; nothing is allocated by the call
    status = torch.full((1,), 99, dtype=torch.int32, device="cuda")
    P.laser_sta_forward_static(b.cfg, *b.args(), out, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return ref, out


def test_static_scratch_entry_point_matches_workspace_entry_point_twice_in_a_row():
    # two different problems back to back: the second call finds the first call's leftovers in the shared array
    w1 = make_custom(U=3, C=7, L=96, d=64, H=4, S=16, M=1, dtype="bf16", seed=41, lengths=[96, 50, 3])
    w2 = make_custom(U=2, C=40, L=128, d=32, H=2, S=32, M=1, dtype="f32", seed=42, lengths=[77, 128], emb_std="one")
    for w in (w1, w2):
        ref, out = _both(w)
        assert err_metric(to_np(out), to_np(ref)) <= TOL[w.spec.dtype]
        assert torch.equal(out, ref)                   # same kernels, same arithmetic: identical bits
        s = w.spec                                     # and against the float64 oracle itself, not only its sibling
        Hp_ref = laser_oracle.sta_forward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, s.S, s.H,
                                          w.gamma)
        assert err_metric(to_np(out), Hp_ref) <= TOL[s.dtype]


def test_static_scratch_rejects_problems_beyond_its_fixed_size():
    w = make_custom(U=1, C=1, L=8, d=32, H=1, S=8, M=1, dtype="f32", seed=1, lengths=[8])
    b = P.DeviceBatch.from_workload(w, path=P.PATH_SIMT)
    big = P.make_config(num_users=64, max_len=4096, d_model=128, d_qk=64, num_heads=4, seg_size=128,
                        num_gsta_layers=0, dtype="f32", total_cands=1, max_cands_per_user=1)
    out = torch.empty((1, 32, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(P.LaserError) as ei:             # rejected on the host before anything is launched
        P.laser_sta_forward_static(big, b.items, b.lengths, b.cands, b.cand_offsets, b.Wq, b.Wk, b.Wv, out)
    assert ei.value.status == -3
