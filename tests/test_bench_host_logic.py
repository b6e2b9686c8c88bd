"""Host-side arithmetic of bench.py (no GPU): algorithmic work counts, roofline entries, and the rule that an ncu
traffic figure is reported only while the kernel's source file is the one the capture was taken from."""
import importlib.util
import os

import numpy as np

from workloads import make_custom

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def _tiny():
    # 2 users: 40 and 7 valid items of width 32, 3 and 2 candidates, segments of 16, 2 heads (d_qk = 32), 2 GSTA layers
    w = make_custom(U=2, C=3, L=48, d=32, H=2, S=16, M=2, dtype="bf16", seed=1, d_qh=16, lengths=[40, 7])
    w.cand_offsets = np.array([0, 3, 5], dtype=np.int32)
    return w


def test_algorithmic_work_counts_valid_items_only():
    b = _bench()
    work = b.algorithmic_work(_tiny())
    d, dqk, H, M = 32, 32, 2, 2
    assert work["valid_items"] == 47 and work["scores"] == 5
    assert work["proj_flops"] == 2 * 47 * d * (dqk + d)                      # K and V of every valid item, once per user
    pairs = 40 * 3 + 7 * 2                                                   # (candidate, valid item) pairs
    assert work["attn_flops"] == 2 * pairs * (dqk + d)                       # scores and gated value sums
    assert work["gate_evals"] == pairs * H
    nseg = [3, 1]                                                            # ceil(40 / 16), ceil(7 / 16)
    assert work["gsta_flops"] == M * (3 * (6 * d * d + 4 * H * nseg[0] * d) + 2 * (6 * d * d + 4 * H * nseg[1] * d))
    assert work["io_bytes"] == (47 * d + 2 * 5 * d) * 2                      # items in, candidates in, z out (bf16)
    assert work["gsta_bytes"] == ((3 * 3 + 2 * 1) * d + 2 * 5 * d) * 2       # every non-empty segment vector once


def test_roofline_entries_divide_work_by_time_and_peak():
    b = _bench()
    w = _tiny()
    peaks = {"hbm_gbs": 1000.0, "bf16_tflops": 100.0, "_source": "measured"}
    work = b.algorithmic_work(w)
    r = b.kernel_roofline(w, "gsta_mma", 0.002, peaks)                       # 2 us
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] == 1000.0 and r["peak_source"] == "of measured"
    assert abs(r["achieved"] - work["gsta_bytes"] / 2e-6 / 1e9) < 1e-9 and abs(r["frac"] - r["achieved"] / 1000.0) < 1e-12
    r = b.kernel_roofline(w, "sta_tc", 0.004, peaks)
    assert r["bound"] == "tensor" and abs(r["achieved"] - work["attn_flops"] / 4e-6 / 1e12) < 1e-12
    assert abs(r["gate_evals_per_s"] - work["gate_evals"] / 4e-6) < 1e-3
    r = b.kernel_roofline(w, "sta_simt", 0.004, dict(peaks, _source="fallback"))
    assert r["bound"] == "alu" and abs(r["peak"] - 148 * 128 * 2 * 1.965e9 / 1e12) < 1e-9 and r["traffic"] is None
    # the projection also carries a bytes-based fraction: 2 d read + 2 (d_qk + d) written per valid item
    r = b.kernel_roofline(w, "tc_proj", 0.001, peaks)
    assert r["bound"] == "tensor" and r["hbm_bytes"] == 47 * 2 * (32 + 32 + 32)
    assert abs(r["hbm_frac"] - r["hbm_bytes"] / 1e-6 / 1e9 / 1000.0) < 1e-12
    # the segment-attention kernel of whichever path ran
    assert b.sta_kernel_roofline(w, {"tc_prep": 0.5, "sta_tc": 0.2, "gsta_mma": 0.3}, peaks)["kernel"] == "sta_tc"
    assert b.sta_kernel_roofline(w, {"stream_pre": 0.1, "stream_sta": 0.2}, peaks)["bound"] == "hbm"
    assert b.sta_kernel_roofline(w, {"gsta_mma": 0.3}, peaks) is None
    # the dominant kernel is the one with the largest time among the step's own kernels
    dom = b.dominant_kernel_roofline(w, {"tc_prep": 0.5, "sta_tc": 0.2, "gsta_mma": 0.3, "fusion": 9.0}, peaks)
    assert dom["kernel"] == "gsta_mma"
    assert b.dominant_kernel_roofline(w, {"tc_prep": 0.5}, peaks) is None


def test_ncu_traffic_is_null_once_the_kernel_source_changed(monkeypatch):
    b = _bench()
    (kernel, workload), (nbytes, digest) = next(iter(b.NCU_TRAFFIC.items()))
    src = b.KERNEL_SOURCE[kernel]
    monkeypatch.setattr(b, "_source_digest", lambda f: digest if f == src else None)
    assert b.ncu_traffic(kernel, workload) == nbytes
    monkeypatch.setattr(b, "_source_digest", lambda f: "0" * 12)
    assert b.ncu_traffic(kernel, workload) is None
    assert b.ncu_traffic("no_such_kernel", workload) is None


def test_parity_figures_report_the_bar_metric_the_raw_error_and_the_error_over_the_signal():
    b = _bench()
    ref = np.array([0.1, -0.2, 4.0, 0.0])
    got = np.array([0.11, -0.2, 4.4, 0.0])
    f = b.parity_figures(got, ref)
    assert abs(f["err"] - 0.1) < 1e-12                   # 0.4 / max(1, 4.0): relative above 1, absolute below
    assert abs(f["max_abs"] - 0.4) < 1e-12
    rms = np.sqrt((0.01 + 0.04 + 16.0) / 4)
    assert abs(f["max_abs_over_rms"] - 0.4 / rms) < 1e-12
    assert b.parity_figures(np.zeros((0, 3)), np.zeros((0, 3))) == {"err": 0.0, "max_abs": 0.0, "max_abs_over_rms": 0.0}


def test_request_batching_ratio_comes_from_the_two_serving_entries():
    b = _bench()
    one = {"workload": "cfg2_serving_bf16", "ms_per_step": 0.04, "value": 1.0e7}
    many = {"workload": "cfg2_serving_bf16_x32_requests", "ms_per_step": 0.1, "value": 1.6e8}
    r = b.request_batching([one, many, {"workload": "cfg4_lifelong_bf16", "ms_per_step": 1.0, "value": 1.0}])
    assert r["speedup"] == 16.0 and r["requests_per_call"] == 32 and abs(r["batched_call_us"] - 100.0) < 1e-9
    assert b.request_batching([one]) is None
