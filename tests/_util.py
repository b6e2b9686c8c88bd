"""Helpers shared by the GPU parity tests (comparison metric, oracle calls, tensor conversion)."""
import numpy as np

from oracle import laser_oracle

TOL = {"f32": 1e-4, "bf16": 2e-2}


def err_metric(got: np.ndarray, ref: np.ndarray) -> float:
    """max_i |g_i - r_i| / max(1, |r_i|): absolute error for small references, relative for large ones."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if got.size == 0:
        return 0.0
    assert np.all(np.isfinite(got)), "non-finite output"
    return float(np.max(np.abs(got - ref) / np.maximum(1.0, np.abs(ref))))


def to_np(t) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def oracle_forward(w, users=None):
    s = w.spec
    return laser_oracle.forward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H,
                                w.gamma, w.tau, users=users)


def cand_rows(w, users):
    rows = []
    for u in users:
        rows.extend(range(int(w.cand_offsets[u]), int(w.cand_offsets[u + 1])))
    return np.array(rows, dtype=np.int64)
