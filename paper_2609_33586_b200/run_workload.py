"""Runs one of the synthetic workloads a few times through the C interface (for profilers and
quick timing):

    python -m paper_2609_33586_b200.run_workload --workload 2 --modes exact,h15 --launches 2

Prints the mean device time per launch of each mode (CUDA events on the launching stream).
"""
from __future__ import annotations

import argparse

import torch

from . import binding
from .inputs import WORKLOADS, make_inputs


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", type=int, default=2, help="index into inputs.WORKLOADS")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (0 = as defined)")
    ap.add_argument("--modes", default="exact,h15")
    ap.add_argument("--launches", type=int, default=2)
    ap.add_argument("--warmup", type=int, default=1)
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]
    if args.batch:
        wl = wl.with_(B=args.batch)
    inp = make_inputs(wl)
    q, k, v = inp.q.cuda(), inp.k.cuda(), inp.v.cuda()
    out = torch.empty((wl.B, wl.Sq, wl.Hq, wl.D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((wl.B, wl.Hq, wl.Sq), dtype=torch.float32, device="cuda")
    binding.device_status_reset()
    for name in args.modes.split(","):
        mode = binding.MODES[name]

        def call():
            binding.attn_fwd(q, k, v, causal=wl.causal, softmax_scale=wl.softmax_scale, weight_mode=mode,
                             q_descale=inp.q_descale, k_descale=inp.k_descale, v_descale=inp.v_descale,
                             out=out, lse=lse)
        for _ in range(args.warmup):
            call()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.launches):
            call()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.launches
        print(f"{wl.name} {name}: {ms * 1e3:.1f} us per launch, {wl.flops / ms / 1e9:.1f} TFLOP/s")
    status = binding.device_status()
    if status != 0:
        raise SystemExit(f"device-side wait expired (status {status:#x})")


if __name__ == "__main__":
    main()
