"""Builds and runs ``csrc/softmax_ceiling.cu``: the softmax arithmetic of the attention kernel in
isolation (scores per clock per SM), the ceiling the SIMT side of the fused kernel can reach.

    python -m paper_2609_33586_b200.softmax_ceiling
"""
from __future__ import annotations

import subprocess
import sys
from pathlib import Path

from .build import CSRC, PKG, _nvcc

EXE = PKG / "softmax_ceiling.bin"


def build() -> Path:
    src = CSRC / "softmax_ceiling.cu"
    deps = [src] + [CSRC / h for h in ("softmax_math.cuh", "weight_map.cuh", "ptx.cuh", "attn_kernel_common.cuh")]
    if EXE.exists() and all(d.stat().st_mtime <= EXE.stat().st_mtime for d in deps):
        return EXE
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-w",
           "-o", str(EXE), str(src)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return EXE


def main() -> int:
    exe = build()
    return subprocess.run([str(exe)]).returncode


if __name__ == "__main__":
    sys.exit(main())
