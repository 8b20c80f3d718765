#!/usr/bin/env python
"""Benchmark of the fused attention forward (Rowmax-H15 vs the exact-exp2 mode of the same kernel).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

A step is one attention forward in h15 mode over one synthetic batch of the headline workload
(causal, 8192 keys, fp8 e4m3 inputs, B=2, 16 heads, D=128).  The same workload is also timed in
exact mode, and its non-causal twin in both modes, for the H15-over-exact speed-up, with the paper's
window protocol (Sec. 5.3, App. B "Measurement protocol and environment").  A matrix of further
workloads (bf16, fp16, head dimension 64, grouped heads, 1K to 32K keys, Rowmax-PoT, the partly
emulated exact control) follows with a lighter protocol; `--matrix none` skips it.  Inputs are
resident in HBM for `value`; the `e2e` figure repeats the step from pinned host buffers with the
copies inside the timed region.  With N > 1 (one process per GPU under torchrun) every rank runs an
independent replica of the workload: the operator has no exchange step.

    python bench.py --workload NAME --modes exact,h15 --launches 2

runs one workload of the matrix a few times and prints its device time (for profilers).
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
from pathlib import Path

import numpy as np
import torch

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2609_33586_b200.inputs import WORKLOADS, Workload, make_inputs, storage_bits  # noqa: E402

HEADLINE = WORKLOADS[2]       # causal 8K fp8
TWIN = WORKLOADS[3]           # non-causal 8K fp8
METRIC = "attn_fwd_tflops_h15_causal_8k_fp8"
# dram__bytes_read.sum + dram__bytes_write.sum of one h15 launch on the headline workload, from the ncu
# capture summarised in profiles/attn_fwd_ws_causal_8k_fp8.txt (algorithmic: 101 MB in + 68 MB out)
NCU_DRAM_BYTES_PER_LAUNCH = 171.1e6 + 32.1e6
# weight mode, or (weight mode, eighths of the scores on the polynomial route) for the partly emulated exact control
MODE_IDS = {"exact": 0, "pot": 1, "h15": 2, "h15k2": 3, "h15k3": 4, "exact_poly": 5,
            "exact_poly_12": (5, 1), "exact_poly_25": (5, 2), "exact_poly_37": (5, 3), "exact_poly_50": (5, 4)}
POLY_SHARE = {"exact_poly": 0.25, "exact_poly_12": 0.125, "exact_poly_25": 0.25, "exact_poly_37": 0.375, "exact_poly_50": 0.5}
N_SMS = 148                   # B200
MUFU_PER_CLK_PER_SM = 16      # ex2 results per clock per SM (Sec. 1)


def matrix_workloads():
    """(name, workload, modes): the timing matrix beside the headline.  Shapes follow the paper's B200 timing
    tables (App. B: batch 1, 16 heads, D = 128, 1K to 32K keys; grouped heads 32/8; FP16; non-causal) and the
    five configurations of the baseline description."""
    paper = lambda name, S, causal, dt, D=128, seed=20: Workload(name, 1, 16, 16, S, S, D, causal, dt, seed)  # noqa: E731
    out = [
        ("causal_8k_bf16", paper("causal_8k_bf16", 8192, True, "bf16"), ("exact", "h15")),
        ("noncausal_8k_bf16", paper("noncausal_8k_bf16", 8192, False, "bf16"), ("exact", "h15")),
        ("causal_8k_fp16", paper("causal_8k_fp16", 8192, True, "fp16"), ("exact", "h15")),
        ("gqa_causal_2k_bf16", WORKLOADS[1], ("exact", "h15")),
        ("causal_16k_gqa_bf16", WORKLOADS[4].with_(name="causal_16k_gqa_bf16"), ("exact", "pot", "h15")),
        ("causal_16k_gqa_fp8", WORKLOADS[4].with_(name="causal_16k_gqa_fp8", in_dtype="fp8_e4m3"), ("exact", "pot", "h15")),
        ("causal_8k_bf16_d64", paper("causal_8k_bf16_d64", 8192, True, "bf16", D=64), ("exact", "h15")),
        ("causal_8k_fp8_d64", paper("causal_8k_fp8_d64", 8192, True, "fp8_e4m3", D=64), ("exact", "h15")),
    ]
    for S in (1024, 2048, 4096, 8192, 16384, 32768):
        nm = f"causal_{S // 1024}k_fp8_b1"
        out.append((nm, paper(nm, S, True, "fp8_e4m3"), ("exact", "h15")))
    out.append(("causal_8k_fp8_family", WORKLOADS[2].with_(name="causal_8k_fp8_family", B=1),
                ("exact", "pot", "h15", "h15k2", "h15k3")))
    # the stronger exact control: a share of the 2^x on the FMA pipe (App. B "FA4's own parameter space")
    out.append(("causal_8k_fp8_emulated_exact", WORKLOADS[2].with_(name="causal_8k_fp8_emulated_exact", B=1),
                ("exact", "exact_poly_12", "exact_poly_25", "exact_poly_37", "exact_poly_50", "h15")))
    out.append(("causal_8k_bf16_emulated_exact", paper("causal_8k_bf16_emulated_exact", 8192, True, "bf16"),
                ("exact", "exact_poly_12", "exact_poly_25", "exact_poly_37", "exact_poly_50", "h15")))
    return out


# ------------------------------------------------------------------------------------------------
# distributed plumbing (timing only; the data path has no collective)
# ------------------------------------------------------------------------------------------------
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value: float, device) -> float:
    """Max of a per-rank scalar over the job (identity without a process group)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU while a timed region runs (NVML through
    pynvml in a thread; nvidia-smi as the fallback)."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self._stop, self._thr = index, [], threading.Event(), None
        self.sm_max = None
        self._nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            self._nvml = pynvml
        except Exception:
            self._nvml = None

    def _sample_nvml(self):
        # the SM clock every time; power and the throttle reasons every fourth time (each query costs about a
        # millisecond, and a timed region may last only a few tens of them)
        n = self._nvml
        sm = float(n.nvmlDeviceGetClockInfo(self._h, n.NVML_CLOCK_SM))
        if len(self.samples) % 4 == 0 or not self.samples:
            pw = n.nvmlDeviceGetPowerUsage(self._h) / 1000.0
            r = n.nvmlDeviceGetCurrentClocksEventReasons(self._h) if hasattr(n, "nvmlDeviceGetCurrentClocksEventReasons") \
                else n.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
            flags = []
            for name, bit in (("hw_slowdown", 0x8), ("sw_power_cap", 0x4), ("sw_thermal_slowdown", 0x20),
                              ("hw_thermal_slowdown", 0x40)):
                if r & bit:
                    flags.append(name)
        else:
            pw, flags = self.samples[-1][1], self.samples[-1][2]
        self.samples.append((sm, pw, flags))

    def _sample_smi(self):
        out = subprocess.run(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                              "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5)
        f = [x.strip() for x in out.stdout.strip().split(",")]
        if len(f) >= 7:
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            flags = [n for i, n in enumerate(names) if f[3 + i].lower().startswith("active")]
            self.sm_max = float(f[1])
            self.samples.append((float(f[0]), float(f[2]), flags))

    def _run(self):
        while not self._stop.is_set():
            try:
                if self._nvml is not None:
                    self._sample_nvml()
                else:
                    self._sample_smi()
            except Exception:
                pass
            self._stop.wait(0.0005 if self._nvml is not None else 0.05)

    def __enter__(self):
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thr.join(timeout=10)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": ["no_samples"]}
        sm = [s[0] for s in self.samples]
        reasons = sorted({f for s in self.samples for f in s[2]})
        return {"sm_mhz": statistics.median(sm), "sm_min_mhz": min(sm), "sm_max_mhz": self.sm_max,
                "power_w_max": max(s[1] for s in self.samples), "samples": len(self.samples),
                "source": "nvml" if self._nvml is not None else "nvidia-smi", "reasons": reasons}


# ------------------------------------------------------------------------------------------------
# CPU oracle legs (the only places this file touches oracle/)
# ------------------------------------------------------------------------------------------------
def sampled_flops(wl: Workload, rows) -> float:
    rows = np.asarray(rows)
    vis = np.minimum(wl.Sk, rows + wl.Sk - wl.Sq + 1) if wl.causal else np.full(rows.shape, wl.Sk)
    return float(4.0 * wl.B * wl.Hq * wl.D * np.maximum(vis, 0).sum())


def oracle_sample(wl: Workload, inp, mode: int, row_stride: int, n_batch=None, n_heads=None):
    """Times the oracle, as it stands, on every `row_stride`-th query row of the first `n_batch`
    batches and `n_heads` kv heads (with their query-head groups) of the workload."""
    from oracle import cpu_oracle as orc
    nb = n_batch or wl.B
    nkv = n_heads or wl.Hkv
    g = wl.Hq // wl.Hkv
    sub = wl.with_(B=nb, Hq=nkv * g, Hkv=nkv)
    rows = np.arange(0, wl.Sq, row_stride, dtype=np.int32)
    q = storage_bits(inp.q[:nb, :, : nkv * g].contiguous())
    k = storage_bits(inp.k[:nb, :, :nkv].contiguous())
    v = storage_bits(inp.v[:nb, :, :nkv].contiguous())
    dt = orc.IN_BF16 if wl.in_dtype == "bf16" else orc.IN_FP8_E4M3
    t0 = time.perf_counter()
    r = orc.attn(q, k, v, in_dtype=dt, causal=wl.causal, softmax_scale=wl.softmax_scale, mode=mode,
                 tile_n=128 if mode != orc.W_EXACT else 0, q_descale=inp.q_descale, k_descale=inp.k_descale,
                 v_descale=inp.v_descale, rows=rows)
    sec = time.perf_counter() - t0
    return {"seconds": sec, "flops": sampled_flops(sub, rows), "threads": r["threads"], "rows": len(rows),
            "pairs": sub.B * sub.Hq}


def cpu_baseline_leg(wl: Workload, inp, row_stride: int = 4):
    s = oracle_sample(wl, inp, MODE_IDS["h15"], row_stride)
    return {"value": s["flops"] / s["seconds"] / 1e12, "unit": "TFLOP/s", "cores": s["threads"], "kind": "oracle",
            "sample": f"every {row_stride}th query row of {wl.name} ({s['rows']} rows x {s['pairs']} (batch, head) "
                      f"pairs, h15 mode, {s['seconds']:.1f} s incl. input decode)"}


def run_reference(args):
    """--impl reference: the CPU oracle on a bounded sample of the same workload, rank 0 only."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    wl = HEADLINE
    inp = make_inputs(wl)
    stride, nb, nh = 64, 1, 4
    for _ in range(args.warmup):
        oracle_sample(wl, inp, MODE_IDS["h15"], stride, nb, nh)
    secs, flops, threads = [], 0.0, 1
    for _ in range(args.steps):
        s = oracle_sample(wl, inp, MODE_IDS["h15"], stride, nb, nh)
        secs.append(s["seconds"]); flops = s["flops"]; threads = s["threads"]
    total = sum(secs)
    value = flops * len(secs) / total / 1e12
    sample = (f"each step = every {stride}th query row of batch 0, heads 0-{nh - 1} of {wl.name}, h15 mode, "
              "oracle as it stands, input decode included")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(secs),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl), "gpu_launches": 0,
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# GPU legs
# ------------------------------------------------------------------------------------------------
def workload_config(wl: Workload):
    return {"workload": wl.name, "B": wl.B, "Hq": wl.Hq, "Hkv": wl.Hkv, "Sq": wl.Sq, "Sk": wl.Sk, "D": wl.D,
            "causal": wl.causal, "in_dtype": wl.in_dtype, "out_dtype": "bf16", "weight_mode": "h15",
            "softmax_scale": wl.softmax_scale, "seed": wl.seed,
            "l2": "Q+K+V+O = 168 MB per step exceeds the 126 MB L2; no explicit flush"}


class DeviceRun:
    def __init__(self, wl: Workload, inp, device):
        from paper_2609_33586_b200 import binding
        self.b, self.wl, self.inp = binding, wl, inp
        self.q, self.k, self.v = (t.to(device) for t in (inp.q, inp.k, inp.v))
        self.o = torch.empty((wl.B, wl.Sq, wl.Hq, wl.D), dtype=torch.bfloat16, device=device)
        self.lse = torch.empty((wl.B, wl.Hq, wl.Sq), dtype=torch.float32, device=device)

    def step(self, mode):
        mode, eighths = mode if isinstance(mode, tuple) else (mode, None)
        self.b.attn_fwd(self.q, self.k, self.v, causal=self.wl.causal, softmax_scale=self.wl.softmax_scale,
                        weight_mode=mode, q_descale=self.inp.q_descale, k_descale=self.inp.k_descale,
                        v_descale=self.inp.v_descale, out=self.o, lse=self.lse, poly_eighths=eighths)

    def time_steps(self, mode: int, steps: int, warmup: int) -> float:
        """ms per step: CUDA events on the launching (current) stream around `steps` back-to-back calls."""
        for _ in range(warmup):
            self.step(mode)
        torch.cuda.synchronize()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            self.step(mode)
        e1.record()
        torch.cuda.synchronize()
        barrier()
        return e0.elapsed_time(e1) / steps


def timed_windows(run: DeviceRun, modes, index: int, device, warmup: int, windows: int, calls: int, rounds: int):
    """The paper's timing protocol (Sec. 5.3; App. B "Measurement protocol and environment"): `warmup` calls per
    mode, then windows of `calls` back-to-back forwards between two CUDA events, `windows` per mode per round,
    the modes in alternating order round by round (forward, reversed, forward, ...); per mode the median of its
    pooled windows.  The SM clock is sampled while each mode's windows run."""
    for name in modes:
        for _ in range(warmup):
            run.step(MODE_IDS[name])
    torch.cuda.synchronize()
    ms = {m: [] for m in modes}
    mhz = {m: [] for m in modes}
    per_round = []
    for r in range(rounds):
        order = list(modes) if r % 2 == 0 else list(reversed(modes))
        got = {}
        for name in order:
            with ClockSampler(index) as smp:
                ws = [max_over_ranks(run.time_steps(MODE_IDS[name], calls, 0), device) for _ in range(windows)]
            ms[name] += ws
            got[name] = statistics.median(ws)
            mhz[name] += [x[0] for x in smp.samples]
        per_round.append(got)
    out = {"protocol": {"warmup_calls": warmup, "windows_per_mode_per_round": windows, "calls_per_window": calls,
                        "rounds": rounds, "order": "alternating"}, "modes": {}}
    for name in modes:
        med = statistics.median(ms[name])
        clk = statistics.median(mhz[name]) if mhz[name] else None
        out["modes"][name] = {"ms": med, "tflops": run.wl.flops / med / 1e9, "sm_mhz_median": clk,
                              "ms_x_mhz": med * clk if clk else None,
                              "ms_min": min(ms[name]), "ms_max": max(ms[name])}
    if "exact" in modes:
        for name in modes:
            if name != "exact":
                out["modes"][name]["speedup_over_exact_pct"] = 100.0 * (out["modes"]["exact"]["ms"] / out["modes"][name]["ms"] - 1.0)
                out["modes"][name]["speedup_pct_per_round"] = [100.0 * (g["exact"] / g[name] - 1.0) for g in per_round]
    return out


def roofline_entries(res, wl: Workload, peaks):
    """Fractions of the roofline per mode: the tensor bound against the measured cuBLAS bf16 rates (burst and
    sustained; fp8 taken as twice bf16, the nominal ratio), and for the exact-like modes also the bound of the
    special-function unit, one ex2 per visible score at 16 per clock per SM at the sampled SM clock; the
    roofline of such a mode is the lower of the two."""
    ratio = 2.0 if wl.in_dtype == "fp8_e4m3" else 1.0
    scores = wl.flops / (4.0 * wl.D)                       # visible (query, key) pairs, by the same convention
    for name, m in res["modes"].items():
        tf = m["tflops"]
        m["frac_tensor_burst"] = tf / (ratio * peaks["bf16_tflops"])
        if peaks.get("bf16_tflops_sustained"):
            m["frac_tensor_sustained"] = tf / (ratio * peaks["bf16_tflops_sustained"])
        if (name == "exact" or name in POLY_SHARE) and m.get("sm_mhz_median"):
            share = 1.0 - POLY_SHARE.get(name, 0.0)         # the emulated share of the scores bypasses the unit
            bound_ms = 1e3 * share * scores / (MUFU_PER_CLK_PER_SM * N_SMS * m["sm_mhz_median"] * 1e6)
            m["mufu_bound_ms"] = bound_ms
            m["frac_mufu"] = bound_ms / m["ms"]
            m["roofline_frac"] = max(m["frac_tensor_burst"], m["frac_mufu"])   # the lower bound in TFLOP/s = the larger fraction
        else:
            m["roofline_frac"] = m["frac_tensor_burst"]
    return res


def energy_leg(run: DeviceRun, index: int, seconds: float):
    """Board energy per forward, the paper's way (App. B "Energy"): a loop of forwards in chunks of 50
    calls, each followed by a synchronisation, while NVML board power is sampled; energy = mean power
    x loop time / forwards completed, no idle power subtracted.  One loop per mode, exact then h15."""
    out = {}
    for name in ("exact", "h15"):
        mode = MODE_IDS[name]
        for _ in range(30):
            run.step(mode)
        torch.cuda.synchronize()
        with ClockSampler(index) as smp:
            t0 = time.perf_counter()
            n = 0
            while time.perf_counter() - t0 < seconds:
                for _ in range(50):
                    run.step(mode)
                torch.cuda.synchronize()
                n += 50
            t1 = time.perf_counter()
        powers = [s[1] for s in smp.samples]
        if not powers or n == 0:
            return None
        skip = min(len(powers) // 10, 50)          # drop the start-up ramp
        mean_w = statistics.mean(powers[skip:])
        sm = statistics.median(s[0] for s in smp.samples)
        out[name] = {"mj_per_forward": 1e3 * mean_w * (t1 - t0) / n, "mean_power_w": mean_w, "forwards": n,
                     "loop_s": t1 - t0, "ms_per_forward": 1e3 * (t1 - t0) / n, "sm_mhz_median": sm}
    out["h15_energy_change_pct"] = 100.0 * (out["h15"]["mj_per_forward"] / out["exact"]["mj_per_forward"] - 1.0)
    out["workload"] = run.wl.name
    return out


def e2e_leg(run: DeviceRun, steps: int, warmup: int):
    """Same step from pinned host buffers: H2D of q, k, v, the kernel, D2H of O and LSE, all on the
    launching stream and inside the timed region."""
    wl, inp = run.wl, run.inp
    hq, hk, hv = (t.contiguous().pin_memory() for t in (inp.q, inp.k, inp.v))
    ho = torch.empty(run.o.shape, dtype=run.o.dtype).pin_memory()
    hl = torch.empty(run.lse.shape, dtype=run.lse.dtype).pin_memory()

    def one():
        run.q.copy_(hq, non_blocking=True); run.k.copy_(hk, non_blocking=True); run.v.copy_(hv, non_blocking=True)
        run.step(MODE_IDS["h15"])
        ho.copy_(run.o, non_blocking=True); hl.copy_(run.lse, non_blocking=True)

    for _ in range(max(1, warmup // 2)):
        one()
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one()
    e1.record()
    torch.cuda.synchronize()
    barrier()
    ms = e0.elapsed_time(e1) / steps
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv))
    d2h = ho.numel() * ho.element_size() + hl.numel() * hl.element_size()
    return ms, h2d, d2h


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {"bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d.get("bf16_tflops_sustained"),
                "hbm_gbs": d["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def run_ours(args):
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention forward has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2609_33586_b200 import binding

    wl = HEADLINE
    inp = make_inputs(wl)
    run = DeviceRun(wl, inp, device)
    binding.device_status_reset()
    peaks = measured_peaks()

    # headline: K steps of the h15 forward, clocks sampled during the region
    with ClockSampler(local_rank) as clk:
        n0 = binding.launch_count()
        ms_h15 = max_over_ranks(run.time_steps(MODE_IDS["h15"], args.steps, args.warmup), device)
        launches = binding.launch_count() - n0 - args.warmup
    clocks = clk.summary()
    # exact mode of the same kernel and the non-causal twin: the paper's window protocol, independent of --steps
    full = dict(warmup=50, windows=7, calls=100, rounds=3)
    sp = roofline_entries(timed_windows(run, ("exact", "h15"), local_rank, device, **full), wl, peaks)
    twin = DeviceRun(TWIN, make_inputs(TWIN), device)
    sp_nc = roofline_entries(timed_windows(twin, ("exact", "h15"), local_rank, device, **full), TWIN, peaks)
    del twin
    energy = energy_leg(run, local_rank, args.energy_seconds) if (world == 1 and args.energy_seconds > 0) else None
    ms_e2e, h2d, d2h = e2e_leg(run, max(3, args.steps // 4), args.warmup)
    ms_e2e = max_over_ranks(ms_e2e, device)
    status = binding.device_status()
    if status != 0:
        raise SystemExit(f"device-side wait expired during the bench (status {status:#x}); numbers invalid")

    # the rest of the timing matrix (lighter protocol: a few seconds per entry)
    matrix = {}
    if args.matrix != "none":
        light = dict(warmup=20, windows=3, calls=30, rounds=3)
        for name, mwl, modes in matrix_workloads():
            if args.matrix not in ("all", name):
                continue
            mrun = DeviceRun(mwl, make_inputs(mwl), device)
            entry = roofline_entries(timed_windows(mrun, modes, local_rank, device, **light), mwl, peaks)
            entry["config"] = {k: v for k, v in workload_config(mwl).items() if k not in ("weight_mode", "l2")}
            matrix[name] = entry
            del mrun
            torch.cuda.empty_cache()
        status = binding.device_status()
        if status != 0:
            raise SystemExit(f"device-side wait expired during the matrix (status {status:#x}); numbers invalid")

    tf = lambda w, ms: world * w.flops / ms / 1e9   # noqa: E731  (TFLOP/s, whole job)
    fp8_peak = 2.0 * peaks["bf16_tflops"]   # dense fp8 : bf16 nominal ratio is 2
    per_gpu = wl.flops / ms_h15 / 1e9
    line = {
        "metric": METRIC, "value": tf(wl, ms_h15), "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_h15, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "fp8_e4m3", "data": "synthetic", "config": workload_config(wl),
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": world * wl.flops / ms_e2e / 1e9, "unit": "TFLOP/s", "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "roofline": {"bound": "tensor", "achieved": per_gpu, "peak": fp8_peak, "unit": "TFLOP/s",
                     "frac": per_gpu / fp8_peak, "traffic": NCU_DRAM_BYTES_PER_LAUNCH,
                     "algorithmic_bytes": float(sum(t.numel() * t.element_size() for t in (run.q, run.k, run.v, run.o, run.lse))),
                     "peak_source": f"2 x {peaks['source']} cuBLAS bf16 burst ({peaks['bf16_tflops']} TFLOP/s); "
                                    "fp8 peak taken as twice the bf16 one (nominal ratio)",
                     "frac_of_nominal_fp8_4500": per_gpu / 4500.0},
        "modes": dict({"causal_8k_fp8": sp, "noncausal_8k_fp8": sp_nc}, **matrix),
    }
    if energy is not None:
        line["energy"] = energy
        # the same step inside a loop of several seconds (power cap active): the sustained end of the headline
        line["value_sustained"] = world * wl.flops / energy["h15"]["ms_per_forward"] / 1e9
        line["roofline"]["frac_sustained"] = (wl.flops / energy["h15"]["ms_per_forward"] / 1e9) / (
            2.0 * (peaks.get("bf16_tflops_sustained") or peaks["bf16_tflops"]))
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline_leg(wl, inp)
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_workload(args):
    """--workload NAME: a few launches of one workload per mode, device time from CUDA events (for profilers)."""
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention forward has no CPU path")
    from paper_2609_33586_b200 import binding
    table = {w.name: w for w in WORKLOADS}
    table.update({n: w for n, w, _ in matrix_workloads()})
    if args.workload not in table:
        raise SystemExit(f"unknown workload {args.workload}; one of {sorted(table)}")
    wl = table[args.workload]
    if args.batch:
        wl = wl.with_(B=args.batch)
    run = DeviceRun(wl, make_inputs(wl), torch.device("cuda", 0))
    binding.device_status_reset()
    for name in args.modes.split(","):
        ms = run.time_steps(MODE_IDS[name], args.launches, max(1, args.warmup_launches))
        print(f"{wl.name} B={wl.B} {name}: {ms * 1e3:.1f} us per launch, {wl.flops / ms / 1e9:.1f} TFLOP/s")
    status = binding.device_status()
    if status != 0:
        raise SystemExit(f"device-side wait expired (status {status:#x})")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the timed CPU oracle leg")
    ap.add_argument("--energy-seconds", type=float, default=4.0,
                    help="length of the energy loop per mode at N=1 (0 = skip)")
    ap.add_argument("--matrix", default="all", help="'all', 'none' or the name of one entry of the timing matrix")
    ap.add_argument("--workload", default=None, help="profiling helper: run only this workload (see --modes, --launches)")
    ap.add_argument("--batch", type=int, default=0, help="with --workload: override the batch size")
    ap.add_argument("--modes", default="exact,h15", help="with --workload: weight modes to run")
    ap.add_argument("--launches", type=int, default=2, help="with --workload: timed launches per mode")
    ap.add_argument("--warmup-launches", type=int, default=1, help="with --workload: untimed launches per mode")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.workload is not None:
        run_workload(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
