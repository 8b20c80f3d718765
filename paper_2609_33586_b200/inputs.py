"""Seeded synthetic inputs for the attention forward.

This module is the only code that the CUDA path's tests, the bench and the CPU oracle's tests
share.  It holds no arithmetic of the method: it draws Gaussian tensors with a seeded CPU
generator, casts them to the storage type and describes the workload shapes.

The shapes follow the paper's B200 timing matrix (batch 1-4, 16 or 32 query heads, grouped
key/value heads, head dimension 128, 4K-16K keys, causal and non-causal, BF16 and FP8 E4M3;
Sec. 5.3 and App. B Table B4) and its 2K model-fidelity shape with 12 query / 2 key-value heads
(App. B Table B2).  The paper's own inputs are fixed-seed synthetic tensors that were not
published, so these stand in for them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np
import torch

E4M3_MAX = 448.0


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    Hq: int
    Hkv: int
    Sq: int
    Sk: int
    D: int
    causal: bool
    in_dtype: str            # "bf16" | "fp16" | "fp8_e4m3"
    seed: int
    peaked_keys: bool = False  # multiply every key row by its own U(0.5, 2) factor

    @property
    def softmax_scale(self) -> float:
        """1/sqrt(D) as the fp32 value the C interface receives."""
        return float(np.float32(1.0 / math.sqrt(self.D)))

    @property
    def flops(self) -> float:
        """4*B*Hq*Sq*Sk*D, halved for a causal mask (the paper's 2 s^2 d convention)."""
        f = 4.0 * self.B * self.Hq * self.Sq * self.Sk * self.D
        return f / 2 if self.causal else f

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations, indexed as in the baseline description (0..4).
WORKLOADS = (
    Workload("tiny_causal_bf16", 1, 2, 2, 256, 256, 64, True, "bf16", 0),
    Workload("gqa_causal_2k_bf16", 4, 12, 2, 2048, 2048, 128, True, "bf16", 1, peaked_keys=True),
    Workload("causal_8k_fp8", 2, 16, 16, 8192, 8192, 128, True, "fp8_e4m3", 2),
    Workload("noncausal_8k_fp8", 2, 16, 16, 8192, 8192, 128, False, "fp8_e4m3", 3),
    Workload("causal_16k_gqa", 1, 32, 8, 16384, 16384, 128, True, "bf16", 4),
)


@dataclass
class Inputs:
    q: torch.Tensor          # (B,Sq,Hq,D) storage dtype, CPU
    k: torch.Tensor          # (B,Sk,Hkv,D)
    v: torch.Tensor
    q_descale: float
    k_descale: float
    v_descale: float


def _to_storage(x: torch.Tensor, in_dtype: str):
    if in_dtype == "bf16":
        return x.to(torch.bfloat16), 1.0
    if in_dtype == "fp16":
        return x.to(torch.float16), 1.0
    if in_dtype == "fp8_e4m3":
        descale = float(np.float32(float(x.abs().max()) / E4M3_MAX))  # the fp32 value the C interface receives
        y = (x / descale).clamp(-E4M3_MAX, E4M3_MAX).to(torch.float8_e4m3fn)
        return y, descale
    raise ValueError(in_dtype)


def make_inputs(w: Workload) -> Inputs:
    """fp32 N(0,1) draws in the order q, k, v from one seeded CPU generator, then the cast."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed)
    q = torch.randn(w.B, w.Sq, w.Hq, w.D, generator=g, dtype=torch.float32)
    k = torch.randn(w.B, w.Sk, w.Hkv, w.D, generator=g, dtype=torch.float32)
    v = torch.randn(w.B, w.Sk, w.Hkv, w.D, generator=g, dtype=torch.float32)
    if w.peaked_keys:
        u = torch.rand(w.B, w.Sk, w.Hkv, 1, generator=g, dtype=torch.float32) * 1.5 + 0.5
        k = k * u
    qs, dq = _to_storage(q, w.in_dtype)
    ks, dk = _to_storage(k, w.in_dtype)
    vs, dv = _to_storage(v, w.in_dtype)
    return Inputs(qs, ks, vs, dq, dk, dv)


def storage_bits(t: torch.Tensor) -> np.ndarray:
    """Raw bit patterns of a bf16 or fp16 (-> uint16) or e4m3 (-> uint8) CPU tensor."""
    t = t.contiguous().cpu()
    if t.dtype == torch.bfloat16 or t.dtype == torch.float16:
        return t.view(torch.int16).numpy().view(np.uint16)
    if t.dtype == torch.float8_e4m3fn:
        return t.view(torch.uint8).numpy()
    raise TypeError(t.dtype)


def weight_map_sweep() -> np.ndarray:
    """fp32 offsets for the weight-map gate: [-150, 0] in steps of 2^-10 (every half-integer and
    quarter-integer tie is on this grid), their fp32 neighbours at the ties, -inf, +-0, and a
    positive stretch (0, 16] in steps of 2^-6."""
    grid = -np.arange(0, 150 * 1024 + 1, dtype=np.float64) / 1024.0
    ties = -np.arange(0, 150 * 4 + 1, dtype=np.float64) / 4.0
    t32 = ties.astype(np.float32)
    near = np.concatenate([np.nextafter(t32, np.float32(-np.inf)), np.nextafter(t32, np.float32(np.inf))])
    pos = np.arange(1, 16 * 64 + 1, dtype=np.float64) / 64.0
    extra = np.array([-np.inf, 0.0, -0.0, -126.0, -126.25, -127.0, -1e30, -3.0e38], dtype=np.float32)
    return np.concatenate([grid.astype(np.float32), near.astype(np.float32),
                           pos.astype(np.float32), extra])


def paper_bit_test_set(seed: int = 0) -> np.ndarray:
    """The bit-level input set described in App. B ("Exponential-map ablation"): 2,000,000 uniform
    draws in [-126, 0], the integers 0..-126 and every multiple of 7*2^-14 in that range
    (2,295,040 points; the multiples contain round-to-nearest-even ties)."""
    rng = np.random.default_rng(seed)
    u = rng.uniform(-126.0, 0.0, size=2_000_000)
    ints = -np.arange(0, 127, dtype=np.float64)
    step = 7.0 / 16384.0
    mult = -np.arange(0, int(126.0 / step) + 1, dtype=np.float64) * step
    return np.concatenate([u, ints, mult]).astype(np.float32)
