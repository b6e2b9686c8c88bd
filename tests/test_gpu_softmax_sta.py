"""GPU parity of the softmax-aggregation STA variant (the paper's ablation of the sigmoid gate) against its oracle."""
import numpy as np
import pytest
import torch

import paper_2602_11562_b200 as P
from oracle import softmax_sta_oracle
from workloads import make_custom
from _util import TOL, err_metric, to_np

pytestmark = pytest.mark.gpu

CASES = [
    dict(U=3, C=5, L=70, d=32, H=2, S=16, M=1, dtype="f32", lengths=[70, 33, 0]),          # ragged, an empty user
    dict(U=2, C=40, L=200, d=64, H=4, S=50, M=1, dtype="f32", lengths=[200, 101]),         # segments of two 32-item chunks
    dict(U=2, C=37, L=1000, d=128, H=2, S=10, M=1, dtype="bf16", lengths=[1000, 437]),     # the paper's production shape
    dict(U=1, C=70, L=96, d=16, H=1, S=96, M=1, dtype="bf16", lengths=[90]),               # one segment, three chunks
    dict(U=4, C=3, L=64, d=24, H=3, S=1, M=1, dtype="f32", lengths=[64, 1, 0, 17]),        # one-item segments: s = v
]


@pytest.mark.parametrize("case", range(len(CASES)))
def test_softmax_sta_matches_oracle(case):
    kw = dict(CASES[case])
    std = "one" if kw["d"] <= 32 else "inv_sqrt_d"
    w = make_custom(seed=800 + case, emb_std=std, **kw)
    s = w.spec
    ref = softmax_sta_oracle.sta_softmax_forward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, s.S, s.H,
                                                 w.gamma)
    b = P.DeviceBatch.from_workload(w)                       # whatever path the config selects: the variant ignores it
    ws = torch.empty(P.laser_sta_softmax_workspace_bytes(b.cfg), dtype=torch.uint8, device="cuda")
    Hp = P.laser_sta_softmax_forward(b.cfg, *b.args(), workspace=ws)
    assert P.laser_check_status(ws) == 0
    e = err_metric(to_np(Hp), ref)
    assert e <= TOL[s.dtype], f"case {case}: err {e}"
    # the sigmoid path on the same inputs is a different function (the gates do not sum to one)
    Hs = P.laser_sta_forward(b.cfg, *b.args())
    if case < 4:
        assert err_metric(to_np(Hs), ref) > 10 * TOL[s.dtype]
