"""Pins for the fusion oracle: explicit loops, a library reduction, special cases and invariants."""
import numpy as np
import torch

from oracle import fusion_oracle


def _case(seed, N_per_user, lengths, Lp, d, S):
    rng = np.random.default_rng(seed)
    U = len(lengths)
    offs = np.concatenate([[0], np.cumsum(N_per_user)]).astype(np.int32)
    N = int(offs[-1])
    Hp = rng.standard_normal((N, Lp, d)) - 0.5            # mostly negative: a zero row would win a careless max
    z = rng.standard_normal((N, d))
    return Hp, z, np.asarray(lengths, dtype=np.int32), offs


def test_fusion_matches_explicit_loops():
    S, Lp, d, r = 4, 5, 3, 3
    Hp, z, lengths, offs = _case(1, [2, 0, 3, 1], [20, 7, 5, 0], Lp, d, S)
    F = fusion_oracle.fusion_forward(Hp, z, lengths, offs, S, r)
    assert F.shape == (6, (2 + r) * d)
    for u in range(4):
        n = min((int(lengths[u]) + S - 1) // S, Lp)
        for c in range(int(offs[u]), int(offs[u + 1])):
            for e in range(d):
                assert F[c, e] == z[c, e]
                best = 0.0
                if n > 0:
                    best = Hp[c, 0, e]
                    for j in range(1, n):
                        if Hp[c, j, e] > best:
                            best = Hp[c, j, e]
                assert F[c, d + e] == best
                for j in range(r):
                    assert F[c, (2 + j) * d + e] == (Hp[c, j, e] if j < n else 0.0)


def test_pooled_part_is_torch_amax_over_the_valid_segments():
    S, Lp, d, r = 8, 6, 16, 2
    Hp, z, lengths, offs = _case(2, [4, 4], [48, 17], Lp, d, S)      # 6 and 3 non-empty segments
    F = fusion_oracle.fusion_forward(Hp, z, lengths, offs, S, r)
    t = torch.from_numpy(Hp)
    np.testing.assert_array_equal(F[:4, d:2 * d], torch.amax(t[:4, :6], dim=1).numpy())
    np.testing.assert_array_equal(F[4:, d:2 * d], torch.amax(t[4:, :3], dim=1).numpy())


def test_one_segment_pool_is_that_segment_and_missing_recent_slots_are_zero():
    S, Lp, d, r = 10, 4, 5, 3
    Hp, z, lengths, offs = _case(3, [3], [9], Lp, d, S)
    F = fusion_oracle.fusion_forward(Hp, z, lengths, offs, S, r)
    np.testing.assert_array_equal(F[:, d:2 * d], Hp[:, 0])
    np.testing.assert_array_equal(F[:, 2 * d:3 * d], Hp[:, 0])
    assert not F[:, 3 * d:].any()


def test_segment_permutation_leaves_the_pool_and_moves_the_recent_slots():
    S, Lp, d, r = 4, 6, 7, 6
    Hp, z, lengths, offs = _case(4, [5], [24], Lp, d, S)
    perm = np.array([3, 0, 5, 1, 4, 2])
    F = fusion_oracle.fusion_forward(Hp, z, lengths, offs, S, r)
    Fp = fusion_oracle.fusion_forward(Hp[:, perm], z, lengths, offs, S, r)
    np.testing.assert_array_equal(F[:, :2 * d], Fp[:, :2 * d])
    np.testing.assert_array_equal(Fp[:, 2 * d:].reshape(5, r, d), F[:, 2 * d:].reshape(5, r, d)[:, perm])
    # each pooled feature is attained by one of the segments and bounds them all
    pooled = F[:, d:2 * d]
    assert (pooled[:, None, :] >= Hp).all() and (pooled[:, None, :] == Hp).any(axis=1).all()
