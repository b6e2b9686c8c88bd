"""Seeded generators for the five benchmark configurations (and small custom ones).

Only input synthesis lives here: random embeddings, ragged lengths, weight
initialisation and rounding of the drawn values to the I/O dtype.  Nothing in
this file evaluates a projection, a gate, an attention score or a softmax.

All floating-point arrays are returned as float32 numpy arrays whose values are
exactly representable in the workload's I/O dtype (bf16 values are a subset of
float32), so a consumer may convert them to bf16 / f32 / f64 without rounding.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Optional

import numpy as np

PAD_SENTINEL = 7.0  # finite, bf16-representable filler for rows at or beyond a user's valid length


@dataclass(frozen=True)
class WorkloadSpec:
    name: str
    U: int                     # users
    C: int                     # candidates per user
    L: int                     # max sequence length (row stride of each user's item block)
    d: int                     # embedding width
    H: int                     # attention heads (STA and GSTA)
    S: int                     # segment size (the paper's w)
    M: int                     # GSTA layers
    dtype: str                 # "f32" or "bf16": dtype of items, candidates, weights and outputs
    seed: int
    d_qh: int = 16             # STA query/key width per head
    emb_std: str = "inv_sqrt_d"  # "one" -> N(0,1); "inv_sqrt_d" -> N(0,1/d)
    length_kind: str = "full"  # full | uniform | lognormal
    len_lo: int = 0
    len_hi: int = 0
    len_median: float = 0.0
    len_sigma: float = 1.0
    dup_frac: float = 0.0      # fraction of valid items that are near-duplicates of one of the user's candidates
    dup_noise: float = 0.3
    tie_wk_to_wq: bool = False
    gamma: Optional[float] = None   # None -> sqrt(d_qh)
    tau: Optional[float] = None     # None -> sqrt(d/H)

    @property
    def d_qk(self) -> int:
        return self.H * self.d_qh

    @property
    def n_seg(self) -> int:
        return -(-self.L // self.S)

    @property
    def N(self) -> int:
        return self.U * self.C


CONFIGS = {
    # Tiny fp32
    "cfg1": WorkloadSpec("cfg1_tiny_f32", U=1, C=16, L=256, d=32, H=1, S=32, M=1, dtype="f32", seed=0,
                         emb_std="one", length_kind="full"),
    # Serving-shaped bf16
    "cfg2": WorkloadSpec("cfg2_serving_bf16", U=1, C=512, L=2048, d=64, H=4, S=64, M=2, dtype="bf16", seed=1,
                         length_kind="uniform", len_lo=1024, len_hi=2048),
    # Batched ranking bf16, 10 % near-duplicates of a candidate
    "cfg3": WorkloadSpec("cfg3_batched_bf16", U=64, C=256, L=4096, d=128, H=4, S=128, M=2, dtype="bf16", seed=2,
                         length_kind="uniform", len_lo=512, len_hi=4096, dup_frac=0.10,
                         tie_wk_to_wq=True, gamma=1.0 / 48.0),
    # Lifelong ultra-long bf16
    "cfg4": WorkloadSpec("cfg4_lifelong_bf16", U=16, C=1024, L=10000, d=64, H=4, S=100, M=2, dtype="bf16", seed=3,
                         length_kind="lognormal", len_lo=100, len_hi=10000, len_median=3000.0, len_sigma=1.0),
    # One candidate per user (memory-bound) bf16
    "cfg5": WorkloadSpec("cfg5_onecand_bf16", U=4096, C=1, L=2048, d=64, H=2, S=64, M=1, dtype="bf16", seed=4,
                         length_kind="uniform", len_lo=256, len_hi=2048),
    # 32 serving-shaped requests (cfg2) handed to the library in ONE call, each request a user of the batch; not one of
    # the five benchmark configurations
    "cfg2x32": WorkloadSpec("cfg2_serving_bf16_x32_requests", U=32, C=512, L=2048, d=64, H=4, S=64, M=2, dtype="bf16",
                            seed=6, length_kind="uniform", len_lo=1024, len_hi=2048),
    # The paper's production shape (experiment set-up: L = 1000, w = 10, 2 heads of d_q = 16, d = 128, two GSTA layers),
    # batched like cfg3; not one of the five benchmark configurations
    "prod": WorkloadSpec("prod_w10_bf16", U=64, C=256, L=1000, d=128, H=2, S=10, M=2, dtype="bf16", seed=5,
                         length_kind="uniform", len_lo=200, len_hi=1000),
}


@dataclass
class Workload:
    spec: WorkloadSpec
    items: np.ndarray          # [U, L, d] float32 (values representable in spec.dtype)
    lengths: np.ndarray        # [U] int32, valid prefix length per user
    cands: np.ndarray          # [N, d] float32
    cand_offsets: np.ndarray   # [U+1] int32, user u owns candidates [off[u], off[u+1])
    Wq: np.ndarray             # [d, d_qk]
    Wk: np.ndarray             # [d, d_qk]
    Wv: np.ndarray             # [d, d]
    Wg: np.ndarray             # [M, 3, d, d]  (q, k, v) per GSTA layer, y = x @ W
    gamma: float
    tau: float
    dup_pos: list = field(default_factory=list)   # per user: (positions, source candidate index) or None

    @property
    def N(self) -> int:
        return int(self.cand_offsets[-1])


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float array to `dtype` ("f32" or "bf16", round-to-nearest-even) and return it as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "f32":
        return x
    if dtype != "bf16":
        raise ValueError(f"unknown dtype {dtype!r}")
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    u += bias
    u &= np.uint32(0xFFFF0000)
    return x


def _xavier_uniform(rng: np.random.Generator, fan_in: int, fan_out: int, shape) -> np.ndarray:
    a = math.sqrt(6.0 / (fan_in + fan_out))
    return rng.uniform(-a, a, size=shape).astype(np.float32)


def _draw_lengths(rng: np.random.Generator, spec: WorkloadSpec) -> np.ndarray:
    if spec.length_kind == "full":
        return np.full(spec.U, spec.L, dtype=np.int32)
    if spec.length_kind == "uniform":
        return rng.integers(spec.len_lo, spec.len_hi + 1, size=spec.U).astype(np.int32)
    if spec.length_kind == "lognormal":
        raw = np.exp(math.log(spec.len_median) + spec.len_sigma * rng.standard_normal(spec.U))
        return np.clip(np.rint(raw), spec.len_lo, spec.len_hi).astype(np.int32)
    raise ValueError(spec.length_kind)


def _generate(spec: WorkloadSpec, lengths: Optional[np.ndarray] = None) -> Workload:
    rng = np.random.Generator(np.random.PCG64(spec.seed))
    U, C, L, d = spec.U, spec.C, spec.L, spec.d
    std = 1.0 if spec.emb_std == "one" else 1.0 / math.sqrt(d)

    # draw order: lengths, items, candidates, W_q, W_k, W_v, GSTA weights
    drawn = _draw_lengths(rng, spec)
    lengths = drawn if lengths is None else np.asarray(lengths, dtype=np.int32)
    assert lengths.shape == (U,) and lengths.min() >= 0 and lengths.max() <= L

    items = rng.standard_normal((U, L, d), dtype=np.float32)
    items *= np.float32(std)
    cands = rng.standard_normal((U * C, d), dtype=np.float32)
    cands *= np.float32(std)

    dup_pos: list = []
    if spec.dup_frac > 0.0:
        for u in range(U):
            ell = int(lengths[u])
            n_dup = int(round(spec.dup_frac * ell))
            if n_dup == 0 or C == 0:
                dup_pos.append(None)
                continue
            pos = rng.choice(ell, size=n_dup, replace=False)
            src = rng.integers(0, C, size=n_dup)
            t = cands[u * C + src].astype(np.float64)
            scale = spec.dup_noise / math.sqrt(d)
            tn = np.linalg.norm(t, axis=1)
            xs = t + rng.standard_normal((n_dup, d)) * scale
            for _attempt in range(16):  # redraw the noise of any duplicate whose cosine is not above 0.9
                cos = np.sum(xs * t, axis=1) / (np.linalg.norm(xs, axis=1) * tn)
                bad = cos <= 0.9
                if not bad.any():
                    break
                xs[bad] = t[bad] + rng.standard_normal((int(bad.sum()), d)) * scale
            assert not bad.any(), "near-duplicate generator could not reach cosine > 0.9"
            items[u, pos] = xs.astype(np.float32)
            dup_pos.append((pos.astype(np.int64), src.astype(np.int64)))

    for u in range(U):
        items[u, int(lengths[u]):] = PAD_SENTINEL

    Wq = _xavier_uniform(rng, d, spec.d_qk, (d, spec.d_qk))
    Wk = _xavier_uniform(rng, d, spec.d_qk, (d, spec.d_qk))
    Wv = _xavier_uniform(rng, d, d, (d, d))
    Wg = _xavier_uniform(rng, d, d, (spec.M, 3, d, d))
    if spec.tie_wk_to_wq:
        Wk = Wq.copy()

    items = round_to_dtype(items, spec.dtype)
    cands = round_to_dtype(cands, spec.dtype)
    Wq, Wk, Wv, Wg = (round_to_dtype(w, spec.dtype) for w in (Wq, Wk, Wv, Wg))

    gamma = float(spec.gamma) if spec.gamma is not None else math.sqrt(spec.d_qh)
    tau = float(spec.tau) if spec.tau is not None else math.sqrt(d / spec.H)
    offs = (np.arange(U + 1, dtype=np.int64) * C).astype(np.int32)
    return Workload(spec, items, lengths, cands, offs, Wq, Wk, Wv, Wg, gamma, tau, dup_pos)


def make_workload(name: str, *, seed_offset: int = 0, users: Optional[int] = None) -> Workload:
    """Build one of the named configurations ("cfg1" .. "cfg5").

    seed_offset: added to the configuration's seed (rank r of a data-parallel run uses seed_offset=r, so
        each rank holds a batch of the same shape and distribution but different values).
    users: generate only the first `users` users' worth of the configuration (a bounded sample of the
        same distribution; the random stream differs from the full configuration's).
    """
    spec = CONFIGS[name]
    if seed_offset:
        spec = replace(spec, seed=spec.seed + 1000 * seed_offset)
    if users is not None and users != spec.U:
        spec = replace(spec, U=int(users), name=f"{spec.name}[users={users}]")
    return _generate(spec)


def make_custom(*, U, C, L, d, H, S, M, dtype="f32", seed=0, d_qh=16, lengths=None, emb_std="inv_sqrt_d",
                gamma=None, tau=None, name="custom") -> Workload:
    """A small custom workload (tests). `lengths` may be an explicit per-user list; default: uniform in [0, L]."""
    spec = WorkloadSpec(name, U=U, C=C, L=L, d=d, H=H, S=S, M=M, dtype=dtype, seed=seed, d_qh=d_qh,
                        emb_std=emb_std, length_kind="uniform", len_lo=0, len_hi=L, gamma=gamma, tau=tau)
    return _generate(spec, lengths=None if lengths is None else np.asarray(lengths, dtype=np.int32))


def make_ffn_weights(d: int, r: int = 4, dtype: str = "bf16", seed: int = 0) -> dict:
    """Seeded weights of the feed-forward refinement (Eq. 6): W1 [d, r d], b1 [r d], W2 [r d, d], b2 [d] and the
    layer norm's gain / shift [d], all rounded to `dtype` and returned as float32 arrays."""
    rng = np.random.Generator(np.random.PCG64(77_000 + seed))
    hid = r * d
    w = {
        "W1": _xavier_uniform(rng, d, hid, (d, hid)),
        "b1": (0.05 * rng.standard_normal(hid)).astype(np.float32),
        "W2": _xavier_uniform(rng, hid, d, (hid, d)),
        "b2": (0.05 * rng.standard_normal(d)).astype(np.float32),
        "ln_g": (1.0 + 0.1 * rng.standard_normal(d)).astype(np.float32),
        "ln_b": (0.1 * rng.standard_normal(d)).astype(np.float32),
    }
    return {k: round_to_dtype(v, dtype) for k, v in w.items()}


def make_gsta_inputs(*, counts, segments, Lp, d, M, seed=0, hp_std=0.5):
    """Seeded inputs for the GSTA stage alone (tests): per user u `counts[u]` candidates whose first `segments[u]` of
    `Lp` segment vectors are non-empty.  Returns (cand_offsets [U+1] int32, Hp [N, Lp, d], cands [N, d],
    Wg [M, 3, d, d]) as float32 arrays of bf16-representable values; rows of empty segments hold NaN (a consumer must
    never use them)."""
    rng = np.random.Generator(np.random.PCG64(55_000 + seed))
    counts = np.asarray(counts, dtype=np.int64)
    offs = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    N = int(offs[-1])
    Hp = (hp_std * rng.standard_normal((N, Lp, d), dtype=np.float32)).astype(np.float32)
    cands = rng.standard_normal((N, d), dtype=np.float32) * np.float32(1.0 / math.sqrt(d))
    Wg = _xavier_uniform(rng, d, d, (M, 3, d, d))
    Hp, cands, Wg = (round_to_dtype(a, "bf16") for a in (Hp, cands, Wg))
    for u, nv in enumerate(segments):
        Hp[int(offs[u]):int(offs[u + 1]), int(nv):, :] = np.float32("nan")
    return offs, Hp, cands, Wg
