"""CPU oracle of LASER's multi-resolution feature fusion (section "Multi-resolution Feature Fusion").

TEST INFRASTRUCTURE ONLY, like the rest of oracle/: imported by tests and the benchmark's checks, never by the CUDA
library or its binding.

The paper lists three views that are concatenated per (user, target): the GSTA output z ("global context"), an
element-wise max pooling of the compact sequence H' ("salient features") and the r most recent segment vectors
s_1 .. s_r ("local recency").  Written out, for a candidate whose user has n non-empty segments:

    F = [ z | max_{j < n} s_j | s_0 | s_1 | ... | s_{r-1} ]        in R^{(2 + r) d}

Readings where the paper is silent (kept identical in the CUDA library):
  * segment 0 holds the most recent items (valid items are a prefix of the sequence, so the tail is missing history);
  * the max runs over the non-empty segments only (a zero row of an empty segment must not beat negative features);
    a user without any segment gets zeros;
  * a recent slot j >= n (or j >= L') is a zero vector.

Pins (tests/test_oracle_fusion.py): explicit Python loops, torch.amax on the valid slice, the one-segment case,
invariance of the pooled part under permutations of the segments.
"""
from __future__ import annotations

import numpy as np


def fusion_forward(Hp, z, lengths, cand_offsets, S, num_recent):
    """Hp [N, L', d], z [N, d] -> F [N, (2 + num_recent) * d] float64."""
    Hp = np.asarray(Hp, dtype=np.float64)
    z = np.asarray(z, dtype=np.float64)
    N, Lp, d = Hp.shape
    r = int(num_recent)
    out = np.zeros((N, (2 + r) * d), dtype=np.float64)
    out[:, :d] = z
    for u in range(len(lengths)):
        a, b = int(cand_offsets[u]), int(cand_offsets[u + 1])
        if b <= a:
            continue
        n = min(-(-int(lengths[u]) // int(S)), Lp)          # non-empty segments of this user
        if n > 0:
            out[a:b, d:2 * d] = Hp[a:b, :n, :].max(axis=1)
        k = min(r, n)
        out[a:b, 2 * d:(2 + k) * d] = Hp[a:b, :k, :].reshape(b - a, k * d)
    return out
