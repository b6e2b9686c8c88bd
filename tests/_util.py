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


def err_figures(got: np.ndarray, ref: np.ndarray) -> dict:
    """The pass/fail metric plus the two figures reported beside it: the raw maximum absolute error and that maximum
    divided by the root mean square of the reference (the error relative to the signal)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if got.size == 0:
        return {"err": 0.0, "max_abs": 0.0, "sum_sq_ref": 0.0, "count": 0}
    assert np.all(np.isfinite(got)), "non-finite output"
    diff = np.abs(got - ref)
    return {"err": float(np.max(diff / np.maximum(1.0, np.abs(ref)))), "max_abs": float(diff.max()),
            "sum_sq_ref": float(np.sum(ref * ref)), "count": int(ref.size)}


def merge_figures(parts) -> dict:
    """Combines err_figures of disjoint parts of a tensor; adds max_abs_over_rms over the whole."""
    parts = [p for p in parts if p["count"] > 0]
    if not parts:
        return {"err": 0.0, "max_abs": 0.0, "max_abs_over_rms": 0.0}
    rms = (sum(p["sum_sq_ref"] for p in parts) / sum(p["count"] for p in parts)) ** 0.5
    max_abs = max(p["max_abs"] for p in parts)
    return {"err": max(p["err"] for p in parts), "max_abs": max_abs, "max_abs_over_rms": max_abs / rms if rms > 0 else 0.0}


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
