"""The paper's analytic cost model (its "Computational Complexity" section), in multiply-accumulates.

TEST INFRASTRUCTURE ONLY.  The paper calls these counts FLOPs; re-deriving its printed totals
shows that one multiply-accumulate counts as one.  Used to pin the work accounting that the
benchmark's roofline figures are built on (which then counts 2 flops per multiply-accumulate).
"""
from __future__ import annotations


def c_proj(L, d, d_q):
    return L * d * d + L * d * d_q            # value projection + low-dimension key projection


def c_attn(L, d, d_q):
    return L * d_q + L * d                    # Q K^T and alpha V for one target


def c_ffn(L, d, w, r):
    return (L / w) * (2 * r * d * d)          # FFN on the compressed sequence only


def c_sta(L, d, d_q, w, r):
    return L * d * (d + d_q) + (L / w) * (2 * r * d * d)      # the paper's rounded total (drops c_attn)


def c_gsta(L, d, w, M):
    return M * (L / w) * (2 * d * d + 2 * d)


def c_laser(L, d, d_q, w, r, M):
    return L * d * d * (1 + d_q / d + (2 * r + 2 * M) / w)


def c_self_attention(L, d):
    return 4 * L * d * d + 2 * L * L * d


def c_target_attention(L, d):
    return 2 * L * d * d + 2 * L * d
