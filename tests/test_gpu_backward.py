"""GPU parity of the backward pass (laser_backward) against its oracle: every gradient, fp32 and bf16 inputs."""
import numpy as np
import pytest
import torch

import paper_2602_11562_b200 as P
from oracle import backward_oracle
from workloads import make_custom

pytestmark = pytest.mark.gpu

# fp32 arithmetic on inputs that are exactly representable (the oracle sees the same bf16-rounded values), sums of up to
# ~1e5 terms finished with atomics: relative to the largest entry of each gradient the error stays far below 1e-4
REL_TO_MAX = 1e-4

CASES = [
    dict(U=3, C=5, L=70, d=32, H=2, S=16, M=2, dtype="f32", lengths=[70, 33, 0]),          # ragged, an empty user
    dict(U=2, C=40, L=200, d=64, H=4, S=50, M=1, dtype="f32", lengths=[200, 101]),         # two chunks per segment
    dict(U=2, C=37, L=300, d=128, H=2, S=10, M=2, dtype="bf16", lengths=[300, 137]),       # production-like segments
    dict(U=1, C=70, L=96, d=16, H=1, S=96, M=3, dtype="bf16", lengths=[90]),               # one segment, three layers
    dict(U=4, C=3, L=64, d=24, H=3, S=1, M=1, dtype="f32", lengths=[64, 1, 0, 17], d_qh=8),  # one-item segments, d_qh = 8
    dict(U=2, C=9, L=40, d=32, H=2, S=8, M=0, dtype="f32", lengths=[40, 13]),              # no GSTA layer: z = t
    dict(U=3, C=130, L=512, d=64, H=4, S=64, M=2, dtype="bf16", lengths=[512, 300, 77]),   # serving-like, more rows
    dict(U=2, C=5, L=40, d=18, H=3, S=8, M=2, dtype="f32", lengths=[40, 21], d_qh=4),      # a width that is no multiple of 4
]


def _check(case_kw, seed, path, bar, want_kernel=None):
    kw = dict(case_kw)
    std = kw.pop("emb_std", "one" if kw["d"] <= 32 else "inv_sqrt_d")
    w = make_custom(seed=seed, emb_std=std, **kw)
    s = w.spec
    rng = np.random.default_rng(seed + 7)
    dz = rng.standard_normal((w.N, s.d)).astype(np.float32)
    ref = backward_oracle.backward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H,
                                   dz.astype(np.float64), w.gamma, w.tau)
    b = P.DeviceBatch.from_workload(w, path=path)
    ws = torch.empty(P.laser_backward_workspace_bytes(b.cfg), dtype=torch.uint8, device="cuda")
    P.laser_profile_enable(True)
    try:
        got = P.laser_backward(b.cfg, *b.args(), b.Wg, torch.from_numpy(dz).cuda(), workspace=ws)
        names = [n for n, _ in P.laser_profile_read()]
    finally:
        P.laser_profile_enable(False)
    assert P.laser_check_status(ws) == 0
    if want_kernel is not None:
        assert ("bwd_sta_mma" in names) == want_kernel, names
    worst = {}
    for k, r in ref.items():
        g = got[k].cpu().numpy().astype(np.float64)
        assert g.shape == r.shape, k
        assert np.isfinite(g).all(), k
        if r.size == 0:                                       # (no GSTA layer: dWg is empty)
            continue
        scale = max(np.max(np.abs(r)), 1e-30)
        worst[k] = np.max(np.abs(g - r)) / scale
        assert worst[k] <= bar, (k, worst[k], scale)
    # padding rows of d_items are exact zeros
    for u in range(s.U):
        assert not got["d_items"][u, int(w.lengths[u]):].any()
    # a second call on the same workspace agrees (the atomically summed parts to rounding, the rest bit for bit).  On the
    # tensor-core path an atomically summed intermediate is then rounded to TF32 as a matrix-product operand, so a
    # last-bit difference of fp32 can become one of 2^-11 in single terms of the weight gradients.
    got2 = P.laser_backward(b.cfg, *b.args(), b.Wg, torch.from_numpy(dz).cuda(), workspace=ws)
    assert torch.equal(got["d_items"], got2["d_items"])
    repeat_bar = 1e-5 if path == P.PATH_SIMT else 2e-4
    for k in ref:
        if ref[k].size:
            diff = (got[k] - got2[k]).abs().max().item()
            assert diff <= repeat_bar * max(np.max(np.abs(ref[k])), 1e-30), k
    return worst


@pytest.mark.parametrize("case", range(len(CASES)))
def test_backward_matches_oracle(case):
    # the FP32-ALU kernels, for either dtype
    _check(CASES[case], 1100 + case, P.PATH_SIMT, REL_TO_MAX, want_kernel=False)


# bf16 batches on the tensor-core kernels.  The operands of the five contractions through the gates are bf16 roundings of
# fp32 intermediates (Q / gamma, K, V, dH', the gates and the score gradients: relative 2^-9 each, `tanh.approx` 2^-11), the
# accumulation is fp32; sums of such terms with random signs stay within a few 1e-3 of the largest entry of a gradient
# (measured: at most 4e-3 on these shapes).  Bar: 2e-2, the forward's bf16 bar.
TENSOR_BAR = 2e-2
TENSOR_CASES = [
    dict(U=3, C=130, L=512, d=64, H=4, S=64, M=2, dtype="bf16", lengths=[512, 300, 77]),   # serving-like (head 16 x 16)
    dict(U=2, C=50, L=512, d=128, H=4, S=128, M=2, dtype="bf16", lengths=[512, 301]),      # batched-ranking-like (16 x 32)
    dict(U=2, C=37, L=300, d=128, H=2, S=10, M=2, dtype="bf16", lengths=[300, 137]),       # production-like (16 x 64, 10-item segments)
    dict(U=2, C=24, L=700, d=64, H=4, S=100, M=1, dtype="bf16", lengths=[700, 455]),       # segments of 100: a 4-row last tile
    dict(U=1, C=70, L=96, d=16, H=1, S=96, M=3, dtype="bf16", lengths=[90]),               # one head, one segment
    dict(U=3, C=9, L=64, d=64, H=2, S=16, M=1, dtype="bf16", lengths=[64, 1, 0], d_qh=32), # d_qh = 32, fewer than 16 candidates
    dict(U=2, C=300, L=128, d=128, H=8, S=32, M=2, dtype="bf16", lengths=[128, 100]),      # eight heads, many candidate tiles
]


@pytest.mark.parametrize("case", range(len(TENSOR_CASES)))
def test_backward_tensor_path_matches_oracle(case):
    worst = _check(TENSOR_CASES[case], 1200 + case, P.PATH_AUTO, TENSOR_BAR, want_kernel=True)
    print("backward tensor path, worst error / largest entry:", {k: f"{v:.2e}" for k, v in worst.items()})


# many segments per user: the attention kernels walk them in chunks of 32 (two and four chunks, ragged last chunk)
MANY_SEGMENTS = [
    dict(U=2, C=9, L=200, d=64, H=4, S=2, M=2, dtype="bf16", lengths=[200, 67]),           # 100 segments, 34 non-empty
    dict(U=2, C=12, L=640, d=128, H=8, S=5, M=1, dtype="bf16", lengths=[640, 333]),        # 128 segments, eight heads
    # (embeddings of variance 1 / d here: with unit variance at this width the GSTA logits reach tens of nats, where the
    # bf16 rounding of the segment vectors alone moves a softmax weight by several per cent)
    dict(U=3, C=8, L=330, d=32, H=2, S=10, M=3, dtype="bf16", lengths=[330, 1, 0], emb_std="inv_sqrt_d"),   # 33 segments
    dict(U=1, C=17, L=1040, d=128, H=2, S=16, M=2, dtype="bf16", lengths=[1029]),          # 65 segments, wide heads
]


@pytest.mark.parametrize("case", range(len(MANY_SEGMENTS)))
def test_backward_tensor_path_many_segments(case):
    _check(MANY_SEGMENTS[case], 1400 + case, P.PATH_AUTO, TENSOR_BAR, want_kernel=True)


@pytest.mark.parametrize("name,users", [("cfg3", (0, 17, 63)), ("cfg2x32", (5, 31)), ("prod", (2, 40)), ("cfg4", (3,))])
def test_backward_full_size_configs_sampled_users(name, users):
    # The batches the benchmark times, in its launch configuration: d_cands and d_items of a user depend on no other user,
    # so the oracle computes those users alone (seconds each); the weight gradients sum over all users and are checked on
    # the small shapes above.
    from workloads import make_workload
    w = make_workload(name)
    s = w.spec
    dz = np.random.default_rng(4242).standard_normal((w.N, s.d)).astype(np.float32)
    ref = backward_oracle.backward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H,
                                   dz.astype(np.float64), w.gamma, w.tau, users=list(users))
    b = P.DeviceBatch.from_workload(w)
    ws = torch.empty(P.laser_backward_workspace_bytes(b.cfg), dtype=torch.uint8, device="cuda")
    got = P.laser_backward(b.cfg, *b.args(), b.Wg, torch.from_numpy(dz).cuda(), workspace=ws)
    assert P.laser_check_status(ws) == 0
    for u in users:
        c0, c1 = int(w.cand_offsets[u]), int(w.cand_offsets[u + 1])
        for g, r, what in ((got["d_cands"][c0:c1], ref["d_cands"][c0:c1], "d_cands"),
                           (got["d_items"][u], ref["d_items"][u], "d_items")):
            g = g.cpu().numpy().astype(np.float64)
            scale = max(float(np.max(np.abs(r))), 1e-30)
            assert np.isfinite(g).all()
            assert np.max(np.abs(g - r)) <= TENSOR_BAR * scale, (name, u, what, float(np.max(np.abs(g - r))), scale)
        assert not got["d_items"][u, int(w.lengths[u]):].any()


def test_backward_of_users_with_few_candidates_keeps_the_fp32_gate_kernels():
    # one candidate per user (the one-candidate serving shape): the matrix products still run on the tensor cores
    kw = dict(U=40, C=1, L=128, d=64, H=2, S=32, M=1, dtype="bf16", lengths=[128] * 20 + [77] * 19 + [0])
    _check(kw, 1300, P.PATH_AUTO, TENSOR_BAR, want_kernel=False)


def test_backward_tensor_path_on_request_only_where_it_exists():
    w = make_custom(U=1, C=4, L=32, d=32, H=2, S=8, M=1, dtype="f32", seed=5)
    b = P.DeviceBatch.from_workload(w, path=P.PATH_TENSOR)
    ws = torch.empty(1 << 24, dtype=torch.uint8, device="cuda")
    with pytest.raises(P.LaserError):
        P.laser_backward(b.cfg, *b.args(), b.Wg, torch.zeros((w.N, 32), device="cuda"), workspace=ws)


def test_backward_rejects_a_short_workspace():
    w = make_custom(U=1, C=4, L=32, d=32, H=2, S=8, M=1, dtype="f32", seed=3)
    b = P.DeviceBatch.from_workload(w)
    ws = torch.empty(P.laser_backward_workspace_bytes(b.cfg) - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(P.LaserError):
        P.laser_backward(b.cfg, *b.args(), b.Wg, torch.zeros((w.N, 32), device="cuda"), workspace=ws)
