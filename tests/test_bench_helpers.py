"""Host-side helpers of bench.py that need no GPU: the timing matrix and the roofline arithmetic."""
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))

import bench  # noqa: E402
from paper_2609_33586_b200.inputs import WORKLOADS  # noqa: E402


def test_matrix_names_are_unique_and_modes_are_known():
    entries = bench.matrix_workloads()
    names = [n for n, _, _ in entries]
    assert len(names) == len(set(names)) and "causal_8k_fp8" not in names      # the headline has its own entry
    for name, wl, modes in entries:
        assert wl.name == name and modes[0] == "exact"
        assert all(m in bench.MODE_IDS for m in modes)
        assert wl.D in (64, 128) and wl.Hq % wl.Hkv == 0
    # the five configurations of the baseline description are all timed somewhere
    shapes = {(w.B, w.Hq, w.Hkv, w.Sq, w.D, w.causal, w.in_dtype) for _, w, _ in entries}
    for cfg in (WORKLOADS[1], WORKLOADS[4], WORKLOADS[4].with_(in_dtype="fp8_e4m3")):
        assert (cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.D, cfg.causal, cfg.in_dtype) in shapes


def test_roofline_fractions():
    wl = WORKLOADS[2]                                   # causal 8K fp8, B = 2, 16 heads: 5.4976e11 flop
    peaks = {"bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0}
    ms = 0.4
    res = {"modes": {"exact": {"ms": ms, "tflops": wl.flops / ms / 1e9, "sm_mhz_median": 2000.0},
                     "exact_poly_25": {"ms": ms, "tflops": wl.flops / ms / 1e9, "sm_mhz_median": 2000.0},
                     "h15": {"ms": ms, "tflops": wl.flops / ms / 1e9, "sm_mhz_median": 2000.0}}}
    out = bench.roofline_entries(res, wl, peaks)["modes"]
    tf = 5.4976e11 / 0.4e-3 / 1e12
    assert out["h15"]["frac_tensor_burst"] == pytest.approx(tf / 3200.0, rel=1e-4)
    assert out["h15"]["frac_tensor_sustained"] == pytest.approx(tf / 2800.0, rel=1e-4)
    assert out["h15"]["roofline_frac"] == out["h15"]["frac_tensor_burst"] and "frac_mufu" not in out["h15"]
    # special-function bound: one ex2 per visible score, 16 per clock per SM, 148 SMs, at the sampled clock
    scores = 2 * 16 * 8192 * 8192 / 2
    bound_ms = 1e3 * scores / (16 * 148 * 2000e6)
    assert out["exact"]["mufu_bound_ms"] == pytest.approx(bound_ms, rel=1e-6)
    assert out["exact"]["frac_mufu"] == pytest.approx(bound_ms / ms, rel=1e-6)
    assert out["exact"]["roofline_frac"] == max(out["exact"]["frac_tensor_burst"], out["exact"]["frac_mufu"])
    assert out["exact_poly_25"]["mufu_bound_ms"] == pytest.approx(0.75 * bound_ms, rel=1e-6)
