"""GPU parity of the fused GSTA kernel alone on large bf16 batches (several thousand candidates: more blocks than run at
once, taken longest first from the order table of the set-up kernel) against the float64 oracle.

The segment vectors are drawn directly (the STA stage is covered elsewhere) and the rows of empty segments hold NaN, so a
row that is used although its segment is empty shows up as a non-finite output."""
import numpy as np
import pytest
import torch

import paper_2602_11562_b200 as P
from oracle import laser_oracle
from workloads import make_gsta_inputs

from _util import TOL, err_metric, to_np

pytestmark = pytest.mark.gpu

CASES = [
    # users x candidates per user, L', d, H, M, S and the valid lengths of the users (cycled)
    dict(U=40, C=128, Lp=32, d=128, H=4, M=2, S=128, lens=[4096, 1, 2048, 2049, 0, 128, 129, 3000, 4095, 640]),
    dict(U=40, C=128, Lp=100, d=64, H=4, M=2, S=100, lens=[10000, 100, 3000, 0, 1601, 9901, 4800, 101]),   # 7 chunks
    dict(U=300, C=17, Lp=32, d=64, H=2, M=1, S=64, lens=[2048, 65, 1000, 1]),          # batches that straddle users
    dict(U=32, C=128, Lp=60, d=128, H=8, M=2, S=16, lens=[960, 17, 500, 0, 959]),      # 8 heads of width 16, 4 chunks
    dict(U=80, C=64, Lp=16, d=128, H=1, M=1, S=8, lens=[128, 127, 8, 64]),             # one chunk, one head
]


def _run(case, uneven=False):
    kw = CASES[case]
    U, Lp, d, H, M, S = kw["U"], kw["Lp"], kw["d"], kw["H"], kw["M"], kw["S"]
    if uneven:
        U = 2 * U                                           # (a seventh of the users will have no candidate)
    lengths = np.array([kw["lens"][u % len(kw["lens"])] for u in range(U)], dtype=np.int32)
    counts = np.full(U, kw["C"], dtype=np.int64)
    if uneven:                                              # users without candidates, uneven counts
        rng = np.random.default_rng(case)
        counts = rng.integers(0, 2 * kw["C"] + 1, size=U)
        counts[::7] = 0
    segs = -(-lengths // S)
    offs, Hp, cands, Wg = make_gsta_inputs(counts=counts, segments=segs, Lp=Lp, d=d, M=M, seed=case)
    N = int(offs[-1])
    L = Lp * S
    tau = float(np.sqrt(d / H))
    z_ref = laser_oracle.gsta_forward(np.nan_to_num(Hp), lengths, offs, cands, Wg, S, H, tau)
    cfg = P.make_config(num_users=U, max_len=L, d_model=d, d_qk=16 * H, num_heads=H, seg_size=S, num_gsta_layers=M,
                        dtype=P.DTYPE_BF16, total_cands=N, max_cands_per_user=int(counts.max()), path=P.PATH_TENSOR)
    ws = torch.empty(P.laser_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    ws.fill_(0xFF)                                           # stale scratch must not matter
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    z = P.laser_gsta_forward(cfg, dev(Hp, torch.bfloat16), dev(lengths, torch.int32), dev(offs, torch.int32),
                             dev(cands, torch.bfloat16), dev(Wg, torch.bfloat16), workspace=ws)
    assert P.laser_check_status(ws) == 0
    e = err_metric(to_np(z), z_ref)
    assert e <= TOL["bf16"], f"z error {e:.3e}"
    return z


@pytest.mark.parametrize("case", range(len(CASES)))
def test_gsta_kernel_alone_large_batches(case):
    _run(case)


@pytest.mark.parametrize("case", [0, 2])
def test_gsta_large_batches_uneven_candidate_counts_and_determinism(case):
    z1 = _run(case, uneven=True)
    z2 = _run(case, uneven=True)
    assert torch.equal(z1, z2)
