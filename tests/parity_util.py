"""Shared helper of the GPU parity tests: run the CUDA path and the CPU oracle on the same seeded
inputs and compare element by element.

Tolerances (absolute): bf16 inputs max 1e-2 and mean 1e-3 on O; fp8 inputs max 5e-2 on O; LSE 1e-3.
In pot and h15 mode a score within 2^-16 (relative) of a rounding boundary may legitimately land on
either side, because the tensor-core fp32 score and the oracle's double score differ in the last
bits; the oracle bounds what such flips can do to a row and the comparison widens the tolerance of
exactly those rows by that bound.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import cpu_oracle as orc
from paper_2609_33586_b200 import binding
from paper_2609_33586_b200.inputs import Inputs, Workload, make_inputs, storage_bits

TIE_EPS = 2.0 ** -16
TOL = {"bf16": {"o_max": 1e-2, "o_mean": 1e-3, "lse": 1e-3},
       "fp16": {"o_max": 1e-2, "o_mean": 1e-3, "lse": 1e-3},
       "fp8_e4m3": {"o_max": 5e-2, "o_mean": None, "lse": 1e-3}}
# Exact mode on fp8 inputs stores P in e4m3 (3 fraction bits, as the paper's baseline kernel does).  On
# causal rows that see fewer than 16 keys two or three comparable weights carry the whole row, their
# rounding (up to 6 % each) does not average out, and |dO| reaches 0.06 for values of magnitude 4-5.
# Those rows get this bound instead of 5e-2; pot and h15 never need it (e5m2 holds their weights exactly).
EXACT_FP8_FEW_KEYS = 16
EXACT_FP8_FEW_KEYS_TOL = 1e-1


def run_cuda(wl: Workload, inp: Inputs, mode: int, device="cuda:0", tau=None, pot_tail=None):
    q, k, v = (t.to(device) for t in (inp.q, inp.k, inp.v))
    o, lse = binding.attn_fwd(q, k, v, causal=wl.causal, softmax_scale=wl.softmax_scale, weight_mode=mode,
                              q_descale=inp.q_descale, k_descale=inp.k_descale, v_descale=inp.v_descale,
                              rescale_tau=tau, pot_tail=pot_tail)
    torch.cuda.synchronize()
    return o, lse


def run_oracle(wl: Workload, inp: Inputs, mode: int, rows=None, tau=None, model_p_storage=False, pot_tail=None):
    dt = {"bf16": orc.IN_BF16, "fp16": orc.IN_FP16, "fp8_e4m3": orc.IN_FP8_E4M3}[wl.in_dtype]
    sch = binding.get_schedule(wl.D, dt, mode, wl.causal)
    if mode == binding.W_EXACT_POLY:
        mode = orc.W_EXACT      # the partly emulated exponential is held to the exact definition
    assert sch["rescale_tau"] == 0.0
    if tau is not None:
        sch["rescale_tau"] = tau
    drop_tail = False
    if pot_tail is not None:
        sch["pot_kmax"], drop_tail = int(pot_tail[0]), bool(pot_tail[1])
    tile = 0 if mode == orc.W_EXACT else sch["tile_n"]   # exact mode: the whole-row definition
    p_kw = {}
    if model_p_storage and sch["p_format"] == binding.P_E4M3:
        # diagnostic reference: the online loop with P rounded to the kernel's e4m3 storage format
        tile = sch["tile_n"]
        p_kw = {"p_round": orc.P_E4M3, "p_off": sch["p_offset_log2"]}
    out = orc.attn(storage_bits(inp.q), storage_bits(inp.k), storage_bits(inp.v), in_dtype=dt,
                    causal=wl.causal, softmax_scale=wl.softmax_scale, mode=mode, tile_n=tile,
                    kv_order=sch["kv_order"], tau=sch["rescale_tau"], kmax=sch["pot_kmax"], drop_tail=drop_tail,
                    q_descale=inp.q_descale, k_descale=inp.k_descale, v_descale=inp.v_descale,
                    tie_eps=TIE_EPS if mode != orc.W_EXACT else 0.0, rows=rows, **p_kw)
    out["modelled_p"] = bool(p_kw)
    return out


def compare(wl: Workload, mode: int, inp: Inputs | None = None, rows=None, device="cuda:0",
            allow_output_rounding: bool = False, tau=None, model_p_storage: bool = False, pot_tail=None):
    """Returns a dict of error statistics; `ok` says whether every gate holds.

    `model_p_storage`: where the kernel stores P in e4m3 (exact mode, and the eighth-octave family
    member, on fp8 inputs) the reference is the oracle's online loop with P rounded to that format.
    Used for inputs with peaked rows, where two or three weights carry a row and their 3-fraction-bit
    rounding shows in O far beyond 5e-2 against the unrounded reference; the standard workloads are
    compared with the unrounded reference.
    `allow_output_rounding` adds half a bf16 ulp of the reference value to the per-row tolerance: O
    is stored in bf16, and for outputs of magnitude 2 and above that rounding alone is 0.008 and
    more.  The standard workloads (N(0,1) values, averaged) do not need it."""
    inp = inp or make_inputs(wl)
    o, lse = run_cuda(wl, inp, mode, device, tau, pot_tail)
    ref = run_oracle(wl, inp, mode, rows, tau, model_p_storage, pot_tail)
    o = o.float().cpu().numpy().transpose(0, 2, 1, 3).astype(np.float64)   # (B,Hq,Sq,D)
    lse = lse.cpu().numpy().astype(np.float64)
    if rows is not None:
        o, lse = o[:, :, rows], lse[:, :, rows]
    tol = TOL[wl.in_dtype]
    err_o = np.abs(o - ref["O"])
    row_err = err_o.max(axis=-1)
    allowed = tol["o_max"] + ref["widen_o"]
    if wl.in_dtype == "fp8_e4m3" and mode in (orc.W_EXACT, binding.W_EXACT_POLY) and wl.causal:
        row_ids = np.arange(wl.Sq) if rows is None else np.asarray(rows)
        few = (row_ids + wl.Sk - wl.Sq + 1) < EXACT_FP8_FEW_KEYS
        allowed = np.where(few[None, None, :], np.maximum(allowed, EXACT_FP8_FEW_KEYS_TOL), allowed)
    if allow_output_rounding:
        allowed = allowed + np.abs(ref["O"]).max(axis=-1) * 2.0 ** -8
    inf_both = np.isneginf(lse) & np.isneginf(ref["LSE"])
    with np.errstate(invalid="ignore"):
        err_l = np.where(inf_both, 0.0, np.abs(lse - ref["LSE"]))
    err_l = np.where(np.isnan(err_l), np.inf, err_l)
    allowed_l = tol["lse"] + ref["widen_lse"]
    clean = ref["nflag"] == 0
    stats = {
        "o_max": float(err_o.max()), "o_mean": float(err_o.mean()),
        "o_max_clean_rows": float(row_err[clean].max()) if clean.any() else 0.0,
        "lse_max": float(err_l.max()),
        "lse_max_clean_rows": float(err_l[clean].max()) if clean.any() else 0.0,
        "rows": int(row_err.size), "tie_rows": int((~clean).sum()), "tie_elems": int(ref["nflag"].sum()),
        "rows_over": int((row_err > allowed).sum()), "lse_over": int((err_l > allowed_l).sum()),
        "nan": int(np.isnan(o).sum()),
    }
    if wl.in_dtype == "fp8_e4m3" and mode in (orc.W_EXACT, binding.W_EXACT_POLY) and wl.causal:
        # reported separately (see EXACT_FP8_FEW_KEYS): the rows under the documented exception and the rest
        stats["o_max_few_key_rows"] = float(row_err[:, :, few].max()) if few.any() else 0.0
        stats["o_max_other_rows"] = float(row_err[:, :, ~few].max()) if (~few).any() else 0.0
    if model_p_storage and ref.get("modelled_p"):
        # the gate above is against the loop with P rounded to the kernel's storage format; the distance to the
        # unrounded reference (the paper's definition) is recorded beside it, not gated
        plain = run_oracle(wl, inp, mode, rows, tau, False, pot_tail)
        stats["o_max_vs_unrounded"] = float(np.abs(o - plain["O"]).max())
        with np.errstate(invalid="ignore"):
            stats["lse_max_vs_unrounded"] = float(np.where(inf_both, 0.0, np.abs(lse - plain["LSE"])).max())
    ok = stats["rows_over"] == 0 and stats["lse_over"] == 0 and stats["nan"] == 0
    if tol["o_mean"] is not None:
        ok = ok and stats["o_mean"] <= tol["o_mean"]
    stats["ok"] = bool(ok)
    return stats
