"""Per-role cycle budget of the fused attention kernel's steady state.

    python -m paper_2609_33586_b200.role_budget [--workload causal_8k_fp8] [--mode h15] [--block 10]

Builds a variant of the library with the in-kernel cycle stamps compiled in (-DROWMAX_TRACE; the
product build has none), runs one forward of the workload (batch 1), and prints, for one CTA, the
mean number of SM clocks between the stamps of the softmax warpgroups, the correction warps and the
MMA warp over the key tiles of its longest work item: what each role spends on which step and how
long the hand-off chain  P written -> P V issued -> next S issued -> S visible  leaves a softmax
warpgroup waiting.
"""
from __future__ import annotations

import argparse
import ctypes
import subprocess
from pathlib import Path

import numpy as np
import torch

from . import binding, build as cuda_build
from .inputs import WORKLOADS, make_inputs

TRACE_LIB = cuda_build.PKG / "libattn_b200_trace.so"


def build_trace_lib() -> Path:
    newest = max((cuda_build.CSRC / f).stat().st_mtime for f in cuda_build.SOURCES + cuda_build.HEADERS)
    if not TRACE_LIB.exists() or TRACE_LIB.stat().st_mtime < newest:
        cmd = [cuda_build._nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
               "-Xcompiler", "-fPIC", "-shared", "-w", "-DROWMAX_TRACE", "-o", str(TRACE_LIB)]
        cmd += [str(cuda_build.CSRC / f) for f in cuda_build.SOURCES] + ["-lcudart"]
        subprocess.run(cmd, check=True)
    return TRACE_LIB


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="causal_8k_fp8")
    ap.add_argument("--mode", default="h15")
    ap.add_argument("--block", type=int, default=10, help="CTA whose roles are stamped")
    args = ap.parse_args()
    binding._LIB_PATH = build_trace_lib()          # this process uses the stamped build
    L = binding.lib()
    L.attn_set_trace.argtypes = [ctypes.c_void_p, ctypes.c_int]
    wl = {w.name: w for w in WORKLOADS}[args.workload].with_(B=1)
    inp = make_inputs(wl)
    q, k, v = inp.q.cuda(), inp.k.cuda(), inp.v.cuda()
    buf = torch.zeros(4 * 64 * 8, dtype=torch.int64, device="cuda")

    def fwd():
        binding.attn_fwd(q, k, v, causal=wl.causal, softmax_scale=wl.softmax_scale, weight_mode=binding.MODES[args.mode],
                         q_descale=inp.q_descale, k_descale=inp.k_descale, v_descale=inp.v_descale)

    for _ in range(3):
        fwd()
    torch.cuda.synchronize()
    L.attn_set_trace(buf.data_ptr(), args.block)
    fwd()
    torch.cuda.synchronize()
    L.attn_set_trace(None, 0)
    if binding.device_status() != 0:
        raise SystemExit("a device-side wait expired")
    t = buf.cpu().numpy().reshape(4, 64, 8).astype(np.float64)
    # Stamps are overwritten by later work items of the CTA; the CTA's first item is its longest (heaviest first), so
    # the tiles of the first item that no later item reaches still hold its stamps: take a run of consecutive tiles
    # whose stamps increase from tile to tile.
    s_full = t[0, :63, 0]
    js = [j for j in range(8, 62) if s_full[j] > 0 and s_full[j + 1] > s_full[j] and s_full[j] > s_full[j - 1]]
    runs, cur = [], []
    for j in js:
        if cur and j != cur[-1] + 1:
            runs.append(cur); cur = []
        cur.append(j)
    runs.append(cur)
    js = max(runs, key=len)[1:-1]
    if len(js) < 4:
        raise SystemExit("too few steady-state tiles stamped; choose another --block")
    j0, j1 = js[0], js[-1]
    sl = slice(j0, j1 + 1)
    nx = slice(j0 + 1, j1 + 2)
    mean = lambda a: float(np.mean(a))   # noqa: E731
    print(f"workload {wl.name} (B=1), mode {args.mode}, CTA {args.block}, key tiles {j0}..{j1} of its first work item; mean SM clocks")
    print(f"period per key tile (both query tiles): {mean(t[0, nx, 0] - t[0, sl, 0]):8.0f}")
    for tt in (0, 1):
        S = t[tt]
        print(f"softmax warpgroup {tt}:")
        print(f"  scores visible -> in registers (tcgen05.ld)      {mean(S[sl, 1] - S[sl, 0]):8.0f}")
        print(f"  row maximum, anchor, rescale factor posted       {mean(S[sl, 2] - S[sl, 1]):8.0f}")
        print(f"  weights, row sum, P written to TMEM              {mean(S[sl, 3] - S[sl, 2]):8.0f}")
        print(f"  store wait, fence, P posted                      {mean(S[sl, 4] - S[sl, 3]):8.0f}")
        print(f"  busy per tile                                    {mean(S[sl, 4] - S[sl, 0]):8.0f}")
        print(f"  waiting for the next scores                      {mean(S[nx, 0] - S[sl, 4]):8.0f}")
        M = t[3][:, 4 * tt:4 * tt + 4]
        print(f"  hand-off chain: P posted -> MMA warp has it      {mean(M[sl, 0] - S[sl, 4]):8.0f}")
        print(f"                  -> P V issued                    {mean(M[sl, 2] - M[sl, 0]):8.0f}")
        print(f"                  -> next S issued                 {mean(M[sl, 3] - M[sl, 2]):8.0f}")
        print(f"                  -> next scores visible           {mean(S[nx, 0] - M[sl, 3]):8.0f}   (P V and S on the tensor cores, commit, wake-up)")
        C = t[2][:, 4 * tt:4 * tt + 3]
        print(f"  correction: factor posted -> seen                {mean(C[sl, 0] - S[sl, 2]):8.0f}")
        print(f"              previous P V complete seen           {mean(C[sl, 1] - C[sl, 0]):8.0f}")
        print(f"              O rescaled (when a row moved), posted{mean(C[sl, 2] - C[sl, 1]):8.0f}")
    ov = np.minimum(t[0, sl, 4], t[1, sl, 4]) - np.maximum(t[0, sl, 0], t[1, sl, 0])
    print(f"both warpgroups busy at the same time, per tile:   {mean(np.maximum(ov, 0)):8.0f}")


if __name__ == "__main__":
    main()
