#!/usr/bin/env python
"""Benchmark of the fused attention forward (Rowmax-H15 vs the exact-exp2 mode of the same kernel).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

A step is one attention forward in h15 mode over one synthetic batch of the headline workload
(causal, 8192 keys, fp8 e4m3 inputs, B=2, 16 heads, D=128).  The same workload is also timed in
exact mode, and its non-causal twin in both modes, for the H15-over-exact speed-up.  Inputs are
resident in HBM for `value`; the `e2e` figure repeats the step from pinned host buffers with the
copies inside the timed region.  With N > 1 (one process per GPU under torchrun) every rank runs an
independent replica of the workload: the operator has no exchange step.
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
NCU_DRAM_BYTES_PER_LAUNCH = 171.8e6 + 32.6e6
MODE_IDS = {"exact": 0, "pot": 1, "h15": 2}


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
        n = self._nvml
        sm = float(n.nvmlDeviceGetClockInfo(self._h, n.NVML_CLOCK_SM))
        pw = n.nvmlDeviceGetPowerUsage(self._h) / 1000.0
        r = n.nvmlDeviceGetCurrentClocksEventReasons(self._h) if hasattr(n, "nvmlDeviceGetCurrentClocksEventReasons") \
            else n.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
        flags = []
        for name, bit in (("hw_slowdown", 0x8), ("sw_power_cap", 0x4), ("sw_thermal_slowdown", 0x20),
                          ("hw_thermal_slowdown", 0x40)):
            if r & bit:
                flags.append(name)
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
            self._stop.wait(0.002 if self._nvml is not None else 0.05)

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

    def step(self, mode: int):
        self.b.attn_fwd(self.q, self.k, self.v, causal=self.wl.causal, softmax_scale=self.wl.softmax_scale,
                        weight_mode=mode, q_descale=self.inp.q_descale, k_descale=self.inp.k_descale,
                        v_descale=self.inp.v_descale, out=self.o, lse=self.lse)

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


def speedup_rounds(run: DeviceRun, steps: int, device, rounds: int = 3):
    """H15-over-exact speed-up as the paper measures it (Sec. 5.3): windows of back-to-back calls
    between two CUDA events, the two modes in alternating order round by round (exact h15 / h15 exact /
    exact h15), speed-up from the medians of each mode's pooled windows; the spread over rounds is
    reported, not a confidence interval."""
    windows = {"exact": [], "h15": []}
    per_round = []
    for r in range(rounds):
        order = ("exact", "h15") if r % 2 == 0 else ("h15", "exact")
        got = {}
        for name in order:
            ms = max_over_ranks(run.time_steps(MODE_IDS[name], steps, 3), device)
            windows[name].append(ms)
            got[name] = ms
        per_round.append(100.0 * (got["exact"] / got["h15"] - 1.0))
    med = {k: statistics.median(v) for k, v in windows.items()}
    return {"exact_ms": med["exact"], "h15_ms": med["h15"],
            "h15_speedup_pct": 100.0 * (med["exact"] / med["h15"] - 1.0),
            "speedup_pct_per_round": per_round, "windows_per_mode": rounds, "calls_per_window": steps}


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
    twin_inp = make_inputs(TWIN)
    twin = DeviceRun(TWIN, twin_inp, device)
    binding.device_status_reset()

    # headline: K steps of the h15 forward, clocks sampled during the region
    with ClockSampler(local_rank) as clk:
        n0 = binding.launch_count()
        ms_h15 = max_over_ranks(run.time_steps(MODE_IDS["h15"], args.steps, args.warmup), device)
        launches = binding.launch_count() - n0 - args.warmup
        # exact mode of the same kernel and the non-causal twin, in alternating rounds
        for _ in range(args.warmup):
            run.step(MODE_IDS["exact"]); twin.step(MODE_IDS["exact"]); twin.step(MODE_IDS["h15"])
        sp = speedup_rounds(run, args.steps, device)
        sp_nc = speedup_rounds(twin, args.steps, device)
    clocks = clk.summary()
    energy = energy_leg(run, local_rank, args.energy_seconds) if (world == 1 and args.energy_seconds > 0) else None
    ms_e2e, h2d, d2h = e2e_leg(run, max(3, args.steps // 4), args.warmup)
    ms_e2e = max_over_ranks(ms_e2e, device)
    status = binding.device_status()
    if status != 0:
        raise SystemExit(f"device-side wait expired during the bench (status {status:#x}); numbers invalid")

    tf = lambda w, ms: world * w.flops / ms / 1e9   # noqa: E731  (TFLOP/s, whole job)
    peaks = measured_peaks()
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
        "modes": {
            "causal_8k_fp8": dict(sp, h15_tflops=tf(wl, sp["h15_ms"]), exact_tflops=tf(wl, sp["exact_ms"])),
            "noncausal_8k_fp8": dict(sp_nc, h15_tflops=tf(TWIN, sp_nc["h15_ms"]), exact_tflops=tf(TWIN, sp_nc["exact_ms"])),
        },
    }
    if energy is not None:
        line["energy"] = energy
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline_leg(wl, inp)
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the timed CPU oracle leg")
    ap.add_argument("--energy-seconds", type=float, default=4.0,
                    help="length of the energy loop per mode at N=1 (0 = skip)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
