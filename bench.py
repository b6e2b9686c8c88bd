#!/usr/bin/env python
"""Benchmark of the STA+GSTA forward pass:  python bench.py --gpus N --steps K --warmup W [--workload cfg3]

One "step" is one laser_forward call (projections, fused segment attention, GSTA) over one batch of seeded
synthetic inputs of a named configuration.  Prints ONE JSON line (rank 0).

  value        user x candidate scores per second, whole job, inputs resident in HBM
  e2e          the same metric through laser_forward_host with pinned HOST buffers (H2D + D2H in the timed region)
  roofline     the dominant kernel's algorithmic work / its CUDA-event duration, against the measured peak
  cpu_baseline the float64 numpy oracle timed on the host cores on a bounded sample of the same workload

--impl reference times the oracle alone (there is no reference implementation to install for this paper).
With torchrun (N > 1) every rank runs the same configuration on its own batch (seed offset = rank); users are
independent, so there is no data-path collective: only the barrier and the max-over-ranks of the device time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "user x candidate scores/sec for STA+GSTA fwd"
UNIT = "scores/s"
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
FALLBACK = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# ----------------------------------------------------------------------------------------------------- helpers
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK)
    p["_source"] = "fallback"
    return p


def algorithmic_work(w):
    """Algorithmic flops / bytes of one step (valid items only; 2 flops per multiply-accumulate)."""
    s = w.spec
    lens = w.lengths.astype(np.int64)
    ncand = (w.cand_offsets[1:] - w.cand_offsets[:-1]).astype(np.int64)
    nseg = -(-lens // s.S)
    esz = 4 if s.dtype == "f32" else 2
    proj = 2 * int(lens.sum()) * s.d * (s.d_qk + s.d)
    attn = 2 * int((lens * ncand).sum()) * (s.d_qk + s.d)
    gates = int((lens * ncand).sum()) * s.H
    gsta = s.M * int((ncand * (6 * s.d * s.d + 4 * s.H * nseg * s.d)).sum())
    io_bytes = (int(lens.sum()) * s.d + 2 * int(ncand.sum()) * s.d) * esz
    gsta_bytes = (int((ncand * nseg).sum()) * s.d + 2 * int(ncand.sum()) * s.d) * esz   # H' rows once, t in, z out
    return {"proj_flops": proj, "attn_flops": attn, "gate_evals": gates, "gsta_flops": gsta, "io_bytes": io_bytes,
            "gsta_bytes": gsta_bytes,
            "valid_items": int(lens.sum()), "scores": int(ncand.sum())}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample(w, budget_users=None, target=4e10):
    """Users forming a bounded sample for the CPU oracle (a prefix of the batch), sized by a rough cost model so
    that the run takes on the order of 10-30 s at the default target (flop-equivalents of numpy float64 work)."""
    s = w.spec
    cost = w.lengths.astype(np.float64) * 0 + s.L  # the oracle projects and gates all L rows of a user
    ncand = (w.cand_offsets[1:] - w.cand_offsets[:-1]).astype(np.float64)
    per_user = cost * (ncand * s.H * 40.0 + s.d * (s.d_qk + s.d) * 2.0) + ncand * s.M * s.n_seg * 4.0 * s.d * s.d
    target = target if budget_users is None else None
    users, acc = [], 0.0
    for u in range(s.U):
        if budget_users is not None and len(users) >= budget_users:
            break
        if target is not None and users and acc + per_user[u] > target:
            break
        users.append(u)
        acc += per_user[u]
    return users


def time_oracle(w, users):
    from oracle import laser_oracle
    s = w.spec
    t0 = time.perf_counter()
    laser_oracle.forward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H, w.gamma, w.tau,
                         users=users, return_hprime=False)
    dt = time.perf_counter() - t0
    scores = int(sum(int(w.cand_offsets[u + 1] - w.cand_offsets[u]) for u in users))
    return dt, scores


def parity_figures(got, ref):
    """The three error figures reported per tensor: the pass/fail metric max |g - r| / max(1, |r|), the raw maximum
    absolute error, and that maximum divided by the root mean square of the reference (error relative to the signal)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if got.size == 0:
        return {"err": 0.0, "max_abs": 0.0, "max_abs_over_rms": 0.0}
    diff = np.abs(got - ref)
    rms = float(np.sqrt(np.mean(ref * ref)))
    return {"err": float(np.max(diff / np.maximum(1.0, np.abs(ref)))), "max_abs": float(diff.max()),
            "max_abs_over_rms": float(diff.max() / rms) if rms > 0 else 0.0}


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


# ----------------------------------------------------------------------------------------------------- arms
def run_reference(args, rank, world):
    """The oracle as it stands, on the host cores; each step is a bounded sample of the workload."""
    if rank != 0:
        return
    from workloads import make_workload
    w = make_workload(args.workload)
    users = oracle_sample(w)
    # shrink the sample so that warmup + steps stay within a few minutes
    dt0, sc0 = time_oracle(w, users[:1])
    per_user = max(dt0, 1e-3)
    budget = 150.0 / max(1, args.steps + args.warmup)
    users = users[:max(1, min(len(users), int(budget / per_user)))]
    for _ in range(args.warmup):
        time_oracle(w, users)
    tot_t, tot_s = 0.0, 0
    for _ in range(args.steps):
        dt, sc = time_oracle(w, users)
        tot_t += dt
        tot_s += sc
    value = tot_s / tot_t
    sample = f"users 0..{len(users) - 1} of {w.spec.U} of {w.spec.name} per step ({tot_s // max(1, args.steps)} scores)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.spec.name, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_cores(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum, bytes per launch) of the main kernels from the ncu
# captures summarised under profiles/, keyed by (kernel, workload).  The kernels of the timed step are captured as they
# run inside one forward call, caches not flushed between them (profiles/dram_traffic_in_sequence_cfg3_cfg5.md); the
# FFN kernel alone, cold.  Each entry names the first 12 hex digits of the SHA-256 of the kernel's source file at capture
# time: once that file changes, the figure is reported as null until the kernel is captured again.
NCU_TRAFFIC = {
    ("sta_tc", "cfg3_batched_bf16"): (117940736, "f31bc8cf77dc"),
    ("tc_proj", "cfg3_batched_bf16"): (57026816, "f31bc8cf77dc"),
    ("gsta_mma", "cfg3_batched_bf16"): (76013824, "b7feccc60e24"),
    ("stream_sta", "cfg5_onecand_bf16"): (626225920, "b1b3c0cd26ca"),
    ("ffn_tc", "cfg3_batched_bf16"): (106956032, "18e4b7d28667"),
}
KERNEL_SOURCE = {"sta_tc": "laser_tensor.cu", "tc_proj": "laser_tensor.cu", "gsta_mma": "laser_gsta.cu",
                 "stream_sta": "laser_stream.cu", "ffn_tc": "laser_ffn.cu"}
OTHER_WORKLOADS = ("cfg1", "cfg2", "cfg2x32", "cfg3", "cfg4", "cfg5", "prod")      # entries of the `configs` array
MAIN_KERNELS = ("sta_tc", "tc_proj", "gsta_mma", "stream_sta",      # kernels of the timed step (roofline candidates)
                "proj_simt_q", "proj_simt_kv", "sta_simt", "gsta_simt")


def _source_digest(fname):
    import hashlib
    path = os.path.join(ROOT, "paper_2602_11562_b200", "csrc", fname)
    try:
        with open(path, "rb") as f:
            return hashlib.sha256(f.read()).hexdigest()[:12]
    except OSError:
        return None


def ncu_traffic(kernel, workload):
    ent = NCU_TRAFFIC.get((kernel, workload))
    if not ent:
        return None
    nbytes, digest = ent
    return nbytes if _source_digest(KERNEL_SOURCE.get(kernel, "")) == digest else None


def kernel_roofline(w, name, ms, peaks):
    """Roofline entry of one kernel: algorithmic work of a launch / its CUDA-event duration, against the measured peak."""
    work = algorithmic_work(w)
    sec = ms * 1e-3
    src = "of measured" if peaks["_source"] == "measured" else "of fallback"
    traffic = ncu_traffic(name, w.spec.name)
    if name.endswith("_simt") or "_simt_" in name:
        # FP32-ALU path (the fp32 configuration): plain FMA arithmetic.  Peak = 148 SMs x 128 FP32 lanes x 2 flops x the
        # maximum SM clock (1965 MHz) = 74.4 TFLOP/s, derived from the unit counts, not measured.
        s = w.spec
        flops = {"proj_simt_q": 2 * w.N * s.d * s.d_qk, "proj_simt_kv": work["proj_flops"], "sta_simt": work["attn_flops"],
                 "gsta_simt": work["gsta_flops"]}.get(name, 0)
        peak = 148 * 128 * 2 * 1.965e9 / 1e12
        achieved = flops / sec / 1e12
        return {"kernel": name, "bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "traffic": None, "peak_source": "derived: 148 SMs x 128 FP32 lanes x 2 x 1.965 GHz",
                "ms": ms}
    if name.startswith("stream") or name.startswith("gsta"):
        nbytes = work["io_bytes"] if name.startswith("stream") else work["gsta_bytes"]
        achieved = nbytes / sec / 1e9
        peak = peaks["hbm_gbs"]
        return {"kernel": name, "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_source": src, "ms": ms,
                "frac_of_nominal": achieved / NOMINAL["hbm_gbs"]}
    flops = work["attn_flops"] if name.startswith("sta") else work["proj_flops"]
    achieved = flops / sec / 1e12
    peak = peaks["bf16_tflops"]
    out = {"kernel": name, "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
           "frac": achieved / peak, "traffic": traffic, "peak_source": src, "ms": ms,
           "frac_of_nominal": achieved / NOMINAL["bf16_tflops"]}
    if name == "tc_proj":
        # the projection moves more than it computes at these widths: 2 d bytes read and 2 (d_qk + d) bytes written per
        # valid item, so its bytes-based fraction is reported beside the flop-based one
        s = w.spec
        nbytes = work["valid_items"] * 2 * (s.d + s.d_qk + s.d)
        out["hbm_bytes"] = nbytes
        out["hbm_achieved_gbs"] = nbytes / sec / 1e9
        out["hbm_frac"] = nbytes / sec / 1e9 / peaks["hbm_gbs"]
    if name.startswith("sta"):
        # the gate (one MUFU tanh per candidate x item x head) is what bounds this kernel: 15.8 / clk / SM measured
        gates = work["gate_evals"] / sec
        out["gate_evals_per_s"] = gates
        out["gate_frac_of_mufu_peak"] = gates / (15.8 * 148 * 1.965e9)
    return out


def sta_kernel_roofline(w, prof, peaks):
    """Roofline entry of the fused segment-attention kernel of the path that ran (the kernel the tensor-peak and
    HBM-bandwidth targets are stated for), or None."""
    for name in ("sta_tc", "stream_sta", "sta_simt"):
        if name in prof:
            return kernel_roofline(w, name, prof[name], peaks)
    return None


def request_batching(entries):
    """Throughput of 32 serving-shaped requests in one call over that of one request per call (from the `configs`
    entries), or None when either was not measured."""
    by = {e["workload"]: e for e in entries}
    one, many = by.get("cfg2_serving_bf16"), by.get("cfg2_serving_bf16_x32_requests")
    if not one or not many:
        return None
    return {"single_request_us": one["ms_per_step"] * 1e3, "requests_per_call": 32,
            "batched_call_us": many["ms_per_step"] * 1e3, "single_scores_per_s": one["value"],
            "batched_scores_per_s": many["value"], "speedup": many["value"] / one["value"]}


def dominant_kernel_roofline(w, prof, peaks):
    """Roofline entry for the kernel with the largest share of the step."""
    main = {k: v for k, v in prof.items() if k in MAIN_KERNELS}
    if not main:
        return None
    name, ms = max(main.items(), key=lambda kv: kv[1])
    return kernel_roofline(w, name, ms, peaks)


def ffn_row(P, w, b, Hp, flush, stream, steps, peaks, dev):
    """Next row of the scope: the feed-forward refinement (Eq. 6, r = 4) of this batch's H', timed on its own (outside
    the step) after a check of sampled rows against the oracle."""
    import torch
    from oracle import ffn_oracle
    from workloads import make_ffn_weights
    s = w.spec
    r = 4
    hid = r * s.d
    need = P.laser_ffn_workspace_bytes(b.cfg, hid)
    if need == 0:
        return None
    fw = make_ffn_weights(s.d, r, s.dtype, seed=0)
    fdev = {k: torch.from_numpy(v).to(b.items.dtype).to(dev) for k, v in fw.items()}
    fws = torch.empty(need, dtype=torch.uint8, device=dev)
    nseg = -(-w.lengths.astype(np.int64) // s.S)
    cpu = np.diff(w.cand_offsets.astype(np.int64))
    rows = int((nseg * cpu).sum())
    # parity on sampled rows (the first and last candidate of up to four users)
    before = {}
    for u in [u for u in range(s.U) if nseg[u] > 0 and cpu[u] > 0][:4]:
        for c in {int(w.cand_offsets[u]), int(w.cand_offsets[u + 1]) - 1}:
            before[c] = (Hp[c, :int(nseg[u])].float().cpu().numpy().astype(np.float64), int(nseg[u]))
    try:
        P.laser_ffn_forward(b.cfg, fdev, Hp, b.lengths, b.cand_offsets, workspace=fws, stream=stream)
    except P.LaserError:
        return None
    assert P.laser_check_status(fws) == 0
    err = 0.0
    for c, (x, n) in before.items():
        ref = ffn_oracle.ffn_rows(x, fw["W1"], fw["b1"], fw["W2"], fw["b2"], fw["ln_g"], fw["ln_b"])
        got = Hp[c, :n].float().cpu().numpy().astype(np.float64)
        err = max(err, float(np.max(np.abs(got - ref) / np.maximum(1.0, np.abs(ref)))))
    tol = 1e-4 if s.dtype == "f32" else 2e-2
    if not (err <= tol):
        raise SystemExit(f"FFN parity failure before timing: error {err:.3e} > {tol}")
    P.laser_profile_enable(True)
    prof = {}
    tot = 0.0
    for _ in range(steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        P.laser_ffn_forward(b.cfg, fdev, Hp, b.lengths, b.cand_offsets, workspace=fws, stream=stream)
        e1.record(stream)
        for name, ms in P.laser_profile_read():
            prof[name] = prof.get(name, 0.0) + ms / steps
        torch.cuda.synchronize()
        tot += e0.elapsed_time(e1) / steps
    P.laser_profile_enable(False)
    # the paper's full compression stack through one call: STA -> Eq. 6 -> GSTA
    z_full = torch.empty((b.cfg.total_cands, s.d), dtype=b.items.dtype, device=dev)
    stack_ms = 0.0
    for i in range(steps + 2):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        P.laser_forward_ffn(b.cfg, *b.args(), b.Wg, fdev, z=z_full, workspace=fws, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        if i >= 2:
            stack_ms += e0.elapsed_time(e1) / steps
    assert P.laser_check_status(fws) == 0
    main = "ffn_tc" if "ffn_tc" in prof else "ffn_simt"
    flops = 4.0 * rows * s.d * hid                       # two products of 2 * d * hid flops per row
    ach = flops / (prof[main] * 1e-3) / 1e12
    peak = peaks["bf16_tflops"]
    return {"kernel": main, "expansion": r, "rows": rows, "ms": tot, "kernels_ms": prof,
            "bound": "tensor" if main == "ffn_tc" else "alu", "achieved": ach, "peak": peak if main == "ffn_tc" else None,
            "unit": "TFLOP/s", "frac": ach / peak if main == "ffn_tc" else None, "flops": flops,
            "traffic": ncu_traffic(main, s.name), "algorithmic_bytes": 2 * rows * s.d * (4 if s.dtype == "f32" else 2),
            "parity": {"err": err, "tol": tol, "rows_checked": sum(n for _, n in before.values())},
            "full_stack": {"call": "laser_forward_ffn", "ms_per_step": stack_ms, "value": w.N / (stack_ms * 1e-3),
                           "unit": UNIT}}


def softmax_row(P, w, b, flush, stream, steps, peaks, dev):
    """Another row of the scope: the softmax-aggregation variant of STA (the paper's ablation of the sigmoid gate) on
    this batch, checked on the first two users with candidates against its oracle, then timed on its own."""
    import torch
    from oracle import softmax_sta_oracle
    s = w.spec
    need = P.laser_sta_softmax_workspace_bytes(b.cfg)
    if need == 0:
        return None
    sws = torch.empty(need, dtype=torch.uint8, device=dev)
    Hs = torch.empty((b.cfg.total_cands, b.cfg.n_seg, s.d), dtype=b.items.dtype, device=dev)
    P.laser_sta_softmax_forward(b.cfg, *b.args(), Hprime=Hs, workspace=sws, stream=stream)
    torch.cuda.synchronize()
    assert P.laser_check_status(sws) == 0
    fig, checked = {"err": 0.0, "max_abs": 0.0, "max_abs_over_rms": 0.0}, 0
    for u in [u for u in range(s.U) if w.cand_offsets[u + 1] > w.cand_offsets[u]][:2]:
        c0, c1 = int(w.cand_offsets[u]), int(w.cand_offsets[u + 1])
        ref = softmax_sta_oracle.sta_softmax_user(w.items[u], w.lengths[u], w.cands[c0:c1], w.Wq, w.Wk, w.Wv, s.S, s.H,
                                                  w.gamma)
        f = parity_figures(Hs[c0:c1].float().cpu().numpy().astype(np.float64), ref)
        fig = {k: max(fig[k], f[k]) for k in fig}
        checked += c1 - c0
    tol = 1e-4 if s.dtype == "f32" else 2e-2
    if not (fig["err"] <= tol):
        raise SystemExit(f"softmax-aggregation parity failure before timing: error {fig['err']:.3e} > {tol}")
    P.laser_profile_enable(True)
    prof, tot = {}, 0.0
    for _ in range(steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        P.laser_sta_softmax_forward(b.cfg, *b.args(), Hprime=Hs, workspace=sws, stream=stream)
        e1.record(stream)
        for name, ms in P.laser_profile_read():
            prof[name] = prof.get(name, 0.0) + ms / steps
        torch.cuda.synchronize()
        tot += e0.elapsed_time(e1) / steps
    P.laser_profile_enable(False)
    main = "sta_tc_softmax" if "sta_tc_softmax" in prof else "sta_simt_softmax"
    work = algorithmic_work(w)
    sec = prof[main] * 1e-3
    out = {"kernel": main, "ms": tot, "kernels_ms": prof, "parity": dict(fig, tol=tol, scores_checked=checked),
           "weight_evals_per_s": work["gate_evals"] / sec}
    if main == "sta_tc_softmax":
        # one MUFU exponential per (candidate, item, head): the same 15.8 / clk / SM bound as the sigmoid gate
        ach = work["attn_flops"] / sec / 1e12
        out.update({"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": ach / peaks["bf16_tflops"],
                    "weight_frac_of_mufu_peak": work["gate_evals"] / sec / (15.8 * 148 * 1.965e9)})
    return out


def backward_row(P, w, b, flush, stream, steps, peaks, dev):
    """Another row of the scope: the backward pass (laser_backward) of this batch for a seeded upstream gradient,
    checked on the first two users with candidates against the backward oracle (their rows of d_cands and d_items
    depend on no other user), then timed on its own.  bf16 batches run on the tensor cores (reported against the measured
    tensor peak scaled to TF32), fp32 batches on the FP32 ALUs (against the derived FP32 peak)."""
    import torch
    from oracle import backward_oracle
    s = w.spec
    need = P.laser_backward_workspace_bytes(b.cfg)
    if need == 0:
        return None
    rng = np.random.default_rng(4242)
    dz = rng.standard_normal((w.N, s.d)).astype(np.float32)
    dz_d = torch.from_numpy(dz).to(dev)
    bws = torch.empty(need, dtype=torch.uint8, device=dev)
    P.laser_profile_enable(True)
    try:
        g = P.laser_backward(b.cfg, *b.args(), b.Wg, dz_d, workspace=bws, stream=stream)
        torch.cuda.synchronize()
        kernels = {}
        for name, ms in P.laser_profile_read():
            kernels[name] = kernels.get(name, 0.0) + ms
    except P.LaserError:
        return None
    finally:
        P.laser_profile_enable(False)
    assert P.laser_check_status(bws) == 0
    tensor = "bwd_gemm_tf32" in kernels
    gates_tensor = "bwd_sta_mma" in kernels
    users = [u for u in range(s.U) if w.cand_offsets[u + 1] > w.cand_offsets[u]][:2]
    ref = backward_oracle.backward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S, s.H,
                                   dz.astype(np.float64), w.gamma, w.tau, users=users)
    err, checked = 0.0, 0
    for u in users:
        c0, c1 = int(w.cand_offsets[u]), int(w.cand_offsets[u + 1])
        for got, want in ((g["d_cands"][c0:c1], ref["d_cands"][c0:c1]), (g["d_items"][u], ref["d_items"][u])):
            want = np.asarray(want)
            scale = max(float(np.max(np.abs(want))), 1e-30)
            err = max(err, float(np.max(np.abs(got.cpu().numpy().astype(np.float64) - want))) / scale)
        checked += c1 - c0
    tol = 2e-2 if tensor else 1e-4        # bf16 operands on the tensor cores / fp32 throughout (tests/test_gpu_backward.py)
    if not (err <= tol):
        raise SystemExit(f"backward parity failure before timing: error {err:.3e} of the largest entry > {tol}")
    del g
    tot = 0.0
    for _ in range(steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        P.laser_backward(b.cfg, *b.args(), b.Wg, dz_d, workspace=bws, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        tot += e0.elapsed_time(e1) / steps
    launches = P.laser_last_launch_count()
    work = algorithmic_work(w)
    # forward recomputed once, then about two products per forward product: three times the forward's flops
    flops = 3.0 * (work["proj_flops"] + 2 * w.N * s.d * s.d_qk + work["attn_flops"] + work["gsta_flops"])
    if tensor:      # matrix products in TF32, gate contractions in bf16: against the TF32 figure (the smaller of the two)
        peak = peaks["bf16_tflops"] * 1.1 / 2.25
        bound, source = "tensor", f"{peaks['_source']} bf16 GEMM peak x nominal tf32 : bf16 ratio (1.1 : 2.25)"
    else:
        peak = 148 * 128 * 2 * 1.965e9 / 1e12
        bound, source = "alu", "derived: 148 SMs x 128 FP32 lanes x 2 x 1.965 GHz"
    ach = flops / (tot * 1e-3) / 1e12
    return {"call": "laser_backward", "ms": tot, "launches": launches, "value": w.N / (tot * 1e-3), "unit": UNIT,
            "bound": bound, "flops": flops, "achieved": ach, "peak": peak, "achieved_unit": "TFLOP/s", "frac": ach / peak,
            "peak_source": source,
            "parity": {"err_over_max": err, "tol": tol, "users_checked": len(users), "scores_checked": checked},
            "matrix_products": "tensor cores (mma.sync, TF32 operands)" if tensor else "FP32 ALUs",
            "gate_contractions": "tensor cores (mma.sync, bf16 operands)" if gates_tensor else "FP32 ALUs",
            "kernel_ms_first_call": {k: round(v, 4) for k, v in sorted(kernels.items())},
            "workspace_bytes": need}


def packed_row(P, w, b, z_padded, ws, flush, stream, steps, dev):
    """Another row of the scope: the same forward on items stored without padding (laser_forward_packed); its z must
    equal the padded layout's bit for bit, and it is timed like the main step."""
    import torch
    s = w.spec
    lens = w.lengths.astype(np.int64)
    offs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    rows = torch.cat([b.items[u, :int(lens[u])] for u in range(s.U)], dim=0) if int(lens.sum()) > 0 else \
        torch.zeros((1, s.d), dtype=b.items.dtype, device=dev)
    rows = rows.contiguous()
    offs_d = torch.from_numpy(offs).to(dev)
    z2 = torch.empty_like(z_padded)
    P.laser_forward_packed(b.cfg, rows, offs_d, b.lengths, b.cands, b.cand_offsets, b.Wq, b.Wk, b.Wv, b.Wg, z=z2,
                           workspace=ws, stream=stream)
    assert P.laser_check_status(ws) == 0
    if not torch.equal(z2, z_padded):
        raise SystemExit("packed layout: z differs from the padded layout's")
    tot = 0.0
    for _ in range(steps):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        P.laser_forward_packed(b.cfg, rows, offs_d, b.lengths, b.cands, b.cand_offsets, b.Wq, b.Wk, b.Wv, b.Wg, z=z2,
                               workspace=ws, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        tot += e0.elapsed_time(e1) / steps
    return {"ms_per_step": tot, "value": w.N / (tot * 1e-3), "unit": UNIT, "item_bytes": int(rows.numel() * rows.element_size()),
            "padded_item_bytes": int(b.items.numel() * b.items.element_size()), "z_identical_to_padded": True}


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist

    import paper_2602_11562_b200 as P
    from workloads import make_workload

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    P.load_library()   # fails loudly if the CUDA library is missing
    peaks = load_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    class _L2Flush:
        """Evicts L2 between timed steps: writes a 256 MB buffer (> 126 MB L2), then reads a second 256 MB buffer so that
        the dirty lines of the write are back in HBM before the timed region starts (otherwise their write-back would be
        charged to the first kernel of the step)."""

        def __init__(self):
            self.a = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
            self.b = torch.zeros(64 << 20, dtype=torch.int32, device=dev)
            self.sink = torch.zeros((), dtype=torch.int64, device=dev)

        def fill_(self, v):
            self.a.fill_(v)
            self.sink += self.b.sum()

    flush = _L2Flush()
    stream = torch.cuda.current_stream()

    def measure(name, steps, oracle_target, sync_ranks, before_timing=None):
        """One configuration: parity of z against the oracle on a bounded sample of users (rank 0, before any timing;
        the same run is the timed CPU baseline), `steps` timed forward calls with an L2 flush before each, and a second
        pass of the same steps with the library's per-kernel CUDA events."""
        w = make_workload(name, seed_offset=rank)
        s = w.spec
        b = P.DeviceBatch.from_workload(w, path=P.PATH_AUTO, device=dev)
        ws = torch.empty(P.laser_workspace_bytes(b.cfg), dtype=torch.uint8, device=dev)
        z = torch.empty((b.cfg.total_cands, s.d), dtype=b.items.dtype, device=dev)

        def step():
            P.laser_forward(b.cfg, *b.args(), b.Wg, z=z, workspace=ws, stream=stream)

        parity = cpu_base = None
        if rank == 0:
            step()
            assert P.laser_check_status(ws) == 0
            users = oracle_sample(w, target=oracle_target)
            from oracle import laser_oracle
            t0 = time.perf_counter()
            _, z_ref = laser_oracle.forward(w.items, w.lengths, w.cands, w.cand_offsets, w.Wq, w.Wk, w.Wv, w.Wg, s.S,
                                            s.H, w.gamma, w.tau, users=users, return_hprime=False)
            dt = time.perf_counter() - t0
            scores = int(sum(int(w.cand_offsets[u + 1] - w.cand_offsets[u]) for u in users))
            rows = np.concatenate([np.arange(int(w.cand_offsets[u]), int(w.cand_offsets[u + 1])) for u in users])
            got = z.float().cpu().numpy().astype(np.float64)[rows]
            tol = 1e-4 if s.dtype == "f32" else 2e-2
            fig = parity_figures(got, z_ref[rows])
            if not (np.isfinite(got).all() and fig["err"] <= tol):
                raise SystemExit(f"parity failure before timing ({s.name}): z error {fig['err']:.3e} > {tol}")
            parity = {"z_err": fig["err"], "z_max_abs": fig["max_abs"], "z_max_abs_over_rms": fig["max_abs_over_rms"],
                      "tol": tol, "users_checked": len(users), "scores_checked": int(rows.size)}
            cpu_base = {"value": scores / dt, "unit": UNIT, "cores": host_cores(), "kind": "oracle",
                        "sample": f"users 0..{len(users) - 1} of {s.U} ({scores} scores) of {s.name}, {dt:.1f} s"}

        for _ in range(max(3, args.warmup)):
            flush.fill_(1)
            step()
        launches = P.laser_last_launch_count()
        if sync_ranks:
            barrier()
        else:
            torch.cuda.synchronize()
        if before_timing:
            before_timing()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for e0, e1 in evs:
            flush.fill_(1)          # evict the previous step's data from L2 (outside the timed bracket)
            e0.record(stream)
            step()
            e1.record(stream)
        if sync_ranks:
            barrier()
        else:
            torch.cuda.synchronize()
        times = [e0.elapsed_time(e1) for e0, e1 in evs]

        # per-kernel durations (CUDA events recorded by the library around each launch), same step, same flush
        P.laser_profile_enable(True)
        prof = {}
        for _ in range(steps):
            flush.fill_(1)
            step()
            for kname, ms in P.laser_profile_read():
                prof[kname] = prof.get(kname, 0.0) + ms / steps
        P.laser_profile_enable(False)
        return {"w": w, "b": b, "ws": ws, "z": z, "times": times, "prof": prof, "parity": parity,
                "cpu_baseline": cpu_base, "launches": launches}

    def summary(m):
        """The per-configuration entry of the `configs` array."""
        w, prof = m["w"], m["prof"]
        mean = sum(m["times"]) / len(m["times"])
        return {"workload": w.spec.name, "value": w.N / (mean * 1e-3), "unit": UNIT, "ms_per_step": mean,
                "ms_per_step_median": statistics.median(m["times"]), "steps": len(m["times"]), "kernels_ms": prof,
                "roofline": dominant_kernel_roofline(w, prof, peaks), "sta_roofline": sta_kernel_roofline(w, prof, peaks),
                "parity": m["parity"], "cpu_baseline": m["cpu_baseline"], "gpu_launches": m["launches"] * len(m["times"])}

    sampler = ClockSampler(local_rank)       # clocks from the start of the timed region to the end of the e2e timing
    head = measure(args.workload, args.steps, 4e10, True, before_timing=sampler.start)
    w, b, ws, z = head["w"], head["b"], head["ws"], head["z"]
    s = w.spec
    step_times = list(head["times"])
    dev_ms = sum(step_times)
    prof = head["prof"]
    parity, cpu_base = head["parity"], head["cpu_baseline"]
    launches_per_step = head["launches"]

    def step():
        P.laser_forward(b.cfg, *b.args(), b.Wg, z=z, workspace=ws, stream=stream)

    # next row of the scope: multi-resolution fusion outputs on the H' and z of this batch (outside the timed step)
    fusion = None
    ffn = None
    packed = None
    softmax = None
    bwd = None
    if rank == 0:
        r_recent = 2
        Hp_full = torch.empty((b.cfg.total_cands, b.cfg.n_seg, s.d), dtype=b.items.dtype, device=dev)
        P.laser_forward(b.cfg, *b.args(), b.Wg, Hprime=Hp_full, z=z, workspace=ws, stream=stream)
        fused = torch.empty((b.cfg.total_cands, (2 + r_recent) * s.d), dtype=b.items.dtype, device=dev)
        fws = torch.zeros(256, dtype=torch.uint8, device=dev)
        fe = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for e0, e1 in fe:
            flush.fill_(1)
            e0.record(stream)
            P.laser_fusion_forward(b.cfg, Hp_full, z, b.lengths, b.cand_offsets, r_recent, fused=fused, workspace=fws,
                                   stream=stream)
            e1.record(stream)
        torch.cuda.synchronize()
        f_ms = sum(e0.elapsed_time(e1) for e0, e1 in fe) / args.steps
        wk = algorithmic_work(w)
        esz = 4 if s.dtype == "f32" else 2
        f_bytes = wk["gsta_bytes"] - wk["scores"] * s.d * esz + wk["scores"] * (2 + r_recent) * s.d * esz
        fusion = {"kernel": "fusion", "num_recent": r_recent, "ms": f_ms, "bound": "hbm",
                  "achieved": f_bytes / (f_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                  "frac": f_bytes / (f_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        del fused
        ffn = ffn_row(P, w, b, Hp_full, flush, stream, args.steps, peaks, dev)
        packed = packed_row(P, w, b, z, ws, flush, stream, args.steps, dev)
        del Hp_full
        softmax = softmax_row(P, w, b, flush, stream, min(args.steps, 10), peaks, dev)
        bwd = backward_row(P, w, b, flush, stream, min(args.steps, 3), peaks, dev)

    # end to end: pinned host buffers in, z out, through laser_forward_host
    hb = P.DeviceBatch.from_workload(w, path=P.PATH_AUTO, device="cpu", pin_host=True)
    hws = torch.empty(P.laser_host_workspace_bytes(hb.cfg), dtype=torch.uint8, device=dev)
    z_h = torch.empty((hb.cfg.total_cands, s.d), dtype=hb.items.dtype).pin_memory()
    # bytes the call moves: every input tensor, except that of the items only each user's valid rows travel when
    # the library finds that cheaper than one copy of the padded array (the library reports what it copies)
    h2d, d2h = P.laser_host_transfer_bytes(hb.cfg, hb.lengths, hb.items)
    h2d_padded = sum(t.numel() * t.element_size() for t in (hb.items, hb.lengths, hb.cands, hb.cand_offsets, hb.Wq,
                                                           hb.Wk, hb.Wv, hb.Wg))
    assert d2h == z_h.numel() * z_h.element_size() and h2d <= h2d_padded
    for _ in range(2):
        P.laser_forward_host(hb.cfg, *hb.args(), hb.Wg, z_h, hws, stream=stream, blocking=True)
    barrier()
    e2e_steps = max(1, min(args.steps, 20))
    ee = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(e2e_steps)]
    for e0, e1 in ee:
        e0.record(stream)
        P.laser_forward_host(hb.cfg, *hb.args(), hb.Wg, z_h, hws, stream=stream, blocking=False)
        e1.record(stream)
    barrier()
    e2e_ms = sum(e0.elapsed_time(e1) for e0, e1 in ee)
    clocks = sampler.stop()

    # the other configurations (one GPU only: each rank of a multi-GPU run times the headline workload alone)
    others = []
    if world == 1 and not args.headline_only:
        del hb, hws, z_h
        del b, ws, z, head
        for name in OTHER_WORKLOADS:
            if name == args.workload:
                continue
            torch.cuda.empty_cache()
            others.append(summary(measure(name, min(args.steps, 20), 4e10, False)))

    if world > 1:
        t = torch.tensor([dev_ms, e2e_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dev_ms, e2e_ms = float(t[0]), float(t[1])
        n_scores = torch.tensor([w.N], dtype=torch.float64, device=dev)
        dist.all_reduce(n_scores)
        total_scores = float(n_scores[0])
    else:
        total_scores = float(w.N)

    if rank == 0:
        ms_per_step = dev_ms / args.steps
        work = algorithmic_work(w)
        roof = dominant_kernel_roofline(w, prof, peaks)
        line = {"metric": METRIC, "value": total_scores / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step,
                "ms_per_step_median": statistics.median(step_times),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32" if s.dtype == "f32" else "bf16", "data": "synthetic",
                "config": {"workload": s.name, "users": s.U, "cands_per_user": s.C, "L": s.L, "d": s.d, "heads": s.H,
                           "d_qk": s.d_qk, "seg_size": s.S, "gsta_layers": s.M, "valid_items": work["valid_items"],
                           "l2": "flushed between timed steps (256 MB write, then 256 MB read so that no dirty lines remain)", "parallelism": f"dp{world} by user"},
                "e2e": {"value": total_scores / (e2e_ms / e2e_steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps,
                        "h2d_bytes_if_padded": h2d_padded},
                "gpu_launches": launches_per_step * args.steps,
                "clocks": clocks,
                "roofline": roof,
                "sta_roofline": sta_kernel_roofline(w, prof, peaks),
                "kernels_ms": prof,
                "fusion": fusion,
                "ffn": ffn,
                "packed_layout": packed,
                "softmax_sta": softmax,
                "backward": bwd,
                "kernel_rooflines": [kernel_roofline(w, k, v, peaks) for k, v in prof.items() if k in MAIN_KERNELS],
                "cpu_baseline": cpu_base,
                "parity": parity,
                "work": work,
                "configs": others,
                "request_batching": request_batching(others)}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg1", "cfg2", "cfg2x32", "cfg3", "cfg4", "cfg5", "prod"],
                    help="the headline configuration (value, roofline, e2e); the others follow in `configs`")
    ap.add_argument("--headline-only", action="store_true", help="skip the `configs` array of the other configurations")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
