"""GPU tests of what stands in for a memory checker and a fault injector: the give-up path of the bounded device-side
waits (exercised by a block that waits for a barrier nothing completes: it gives up by construction, nothing faults or
hangs) and the untouched gaps between the workspace regions after a call on every path."""
import numpy as np
import pytest
import torch

import paper_2602_11562_b200 as P
from workloads import make_custom, make_ffn_weights

from _util import TOL, err_metric, oracle_forward, to_np

pytestmark = pytest.mark.gpu


def test_bounded_wait_gives_up_reports_timeout_and_leaves_the_context_usable():
    w = make_custom(U=2, C=150, L=256, d=64, H=4, S=64, M=2, dtype="bf16", seed=21, lengths=[256, 77])
    b = P.DeviceBatch.from_workload(w, path=P.PATH_TENSOR)
    ws = torch.empty(P.laser_workspace_bytes(b.cfg), dtype=torch.uint8, device="cuda")
    _, z_ref = oracle_forward(w)
    for poll_limit in (64, 1024):
        P.laser_selftest_wait_timeout(ws, poll_limit)
        assert P.laser_check_status(ws) == -5
        assert P.laser_status_string(-5) == "a bounded device-side wait gave up"
        # the same workspace, right after: a clean forward (tensor memory was released, the status word is cleared)
        z = P.laser_forward(b.cfg, *b.args(), b.Wg, workspace=ws)
        assert P.laser_check_status(ws) == 0
        assert err_metric(to_np(z), z_ref) <= TOL["bf16"]
    with pytest.raises(P.LaserError):
        P.laser_selftest_wait_timeout(ws, 0)
    with pytest.raises(P.LaserError):
        P.laser_selftest_wait_timeout(ws, 1 << 20)             # the budget itself is bounded


def _outside_regions(cfg, nbytes):
    keep = np.ones(nbytes, dtype=bool)
    for off, size in P.laser_workspace_regions(cfg):
        keep[off:off + size] = False
    return torch.from_numpy(keep)


CASES = {
    "simt": dict(U=3, C=37, L=96, d=64, H=4, S=24, M=2, dtype="bf16", lengths=[0, 96, 41]),
    "tensor": dict(U=3, C=200, L=512, d=64, H=4, S=64, M=2, dtype="bf16", lengths=[512, 301, 0]),
    "stream": dict(U=70, C=1, L=300, d=64, H=2, S=64, M=1, dtype="bf16", lengths=None),
}


@pytest.mark.parametrize("path", ["simt", "tensor", "stream"])
def test_no_kernel_writes_outside_the_workspace_regions(path):
    w = make_custom(seed=31, **CASES[path])
    b = P.DeviceBatch.from_workload(w, path={"simt": P.PATH_SIMT, "tensor": P.PATH_TENSOR, "stream": P.PATH_STREAM}[path])
    nbytes = P.laser_workspace_bytes(b.cfg)
    outside = _outside_regions(b.cfg, nbytes).cuda()
    assert int(outside.sum()) >= 256 * len(P.laser_workspace_regions(b.cfg))
    ws = torch.full((nbytes,), 0xA5, dtype=torch.uint8, device="cuda")
    Hp, z = P.laser_forward(b.cfg, *b.args(), b.Wg, workspace=ws, want_hprime=True)
    assert P.laser_check_status(ws) == 0
    z2 = P.laser_forward(b.cfg, *b.args(), b.Wg, workspace=ws)       # H' in the internal buffer this time
    assert P.laser_check_status(ws) == 0 and torch.equal(z, z2)
    assert bool((ws[outside] == 0xA5).all()), "a kernel wrote outside the regions of the workspace carve-up"
    _, z_ref = oracle_forward(w)
    assert err_metric(to_np(z), z_ref) <= TOL["bf16"]


def test_no_kernel_writes_outside_the_workspace_regions_ffn():
    w = make_custom(seed=32, **CASES["tensor"])
    s = w.spec
    b = P.DeviceBatch.from_workload(w, path=P.PATH_TENSOR)
    fw = make_ffn_weights(s.d, 4, "bf16", seed=5)
    fdev = {k: torch.from_numpy(v).to(torch.bfloat16).cuda() for k, v in fw.items()}
    nbytes = P.laser_ffn_workspace_bytes(b.cfg, 4 * s.d)
    main = P.laser_workspace_bytes(b.cfg)
    outside = _outside_regions(b.cfg, nbytes)
    outside[main:] = False                                 # the feed-forward kernels' own scratch follows the main workspace
    outside = outside.cuda()
    ws = torch.full((nbytes,), 0xA5, dtype=torch.uint8, device="cuda")
    P.laser_forward_ffn(b.cfg, *b.args(), b.Wg, fdev, workspace=ws)
    assert P.laser_check_status(ws) == 0
    assert bool((ws[outside] == 0xA5).all()), "a kernel wrote outside the regions of the workspace carve-up"
