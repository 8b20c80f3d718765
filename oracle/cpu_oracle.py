"""ctypes front end of the CPU oracle (``attn_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the bench's CPU-baseline legs may import this module; the
product package never does.  It compiles ``attn_oracle.c`` with gcc on first use (``build()``)
and marshals NumPy arrays to the C functions.  No arithmetic of the method lives here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "attn_oracle.c"
_LIB = _HERE / "liboracle.so"

W_EXACT, W_POT, W_H15, W_H15K2, W_H15K3 = 0, 1, 2, 3, 4
IN_BF16, IN_FP8_E4M3, IN_FP16 = 0, 1, 2
P_NONE, P_BF16, P_E4M3, P_E5M2 = 0, 1, 2, 3

_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle into ``liboracle.so`` next to its source (gcc, -O2, OpenMP)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=gnu11", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
               "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(str(build()))
        L.oracle_decode_bf16.restype = ctypes.c_double
        L.oracle_decode_bf16.argtypes = [ctypes.c_uint16]
        L.oracle_decode_fp16.restype = ctypes.c_double
        L.oracle_decode_fp16.argtypes = [ctypes.c_uint16]
        L.oracle_decode_e4m3.restype = ctypes.c_double
        L.oracle_decode_e4m3.argtypes = [ctypes.c_uint8]
        L.oracle_weight_map.restype = ctypes.c_int
        L.oracle_weight_map.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                                        ctypes.c_int, ctypes.c_int, ctypes.c_int]
        L.oracle_p_round.restype = ctypes.c_double
        L.oracle_p_round.argtypes = [ctypes.c_double, ctypes.c_int, ctypes.c_int]
        L.oracle_attn.restype = ctypes.c_int
        L.oracle_attn.argtypes = (
            [ctypes.c_void_p] * 3 + [ctypes.c_int] * 8 + [ctypes.c_float] * 4
            + [ctypes.c_int] * 3 + [ctypes.c_double] + [ctypes.c_int] * 4 + [ctypes.c_double]
            + [ctypes.c_void_p, ctypes.c_int] + [ctypes.c_void_p] * 5 + [ctypes.c_int])
        _lib = L
    return _lib


def decode_bf16(bits: int) -> float:
    return lib().oracle_decode_bf16(int(bits))


def decode_fp16(bits: int) -> float:
    return lib().oracle_decode_fp16(int(bits))


def decode_e4m3(bits: int) -> float:
    return lib().oracle_decode_e4m3(int(bits))


def p_round(w: float, fmt: int, p_off: int = 0) -> float:
    """The P-storage diagnostic on one weight: w * 2^p_off rounded to ``fmt``, divided by 2^p_off."""
    return lib().oracle_p_round(float(w), fmt, p_off)


def weight_map(x, mode: int, kmax: int = 20, drop_tail: bool = False) -> np.ndarray:
    """Weights (float64) of the fp32 offsets ``x`` under ``mode`` (``kmax``, ``drop_tail``: Rowmax-PoT only)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    w = np.empty(x.shape, dtype=np.float64)
    rc = lib().oracle_weight_map(x.ctypes.data, w.ctypes.data, x.size, mode, kmax, int(drop_tail))
    if rc != 0:
        raise ValueError(f"oracle_weight_map failed: {rc}")
    return w


def attn(q, k, v, *, in_dtype: int, causal: bool, softmax_scale: float, mode: int,
         tile_n: int = 0, kv_order: int = 1, tau: float = 0.0, kmax: int = 20, drop_tail: bool = False,
         q_descale: float = 1.0, k_descale: float = 1.0, v_descale: float = 1.0,
         p_round: int = P_NONE, p_off: int = 0, tie_eps: float = 0.0, rows=None,
         nthreads: int = 0):
    """Attention forward on raw storage arrays.

    ``q`` is (B,Sq,Hq,D) and ``k``/``v`` are (B,Sk,Hkv,D): uint16 arrays holding bf16 (or, with IN_FP16, IEEE half) bit patterns,
    or uint8 arrays holding e4m3 bit patterns.  Returns a dict with ``O`` (B,Hq,R,D) and ``LSE``
    (B,Hq,R) in float64 over the R requested query rows, the tie bookkeeping arrays, and the
    number of threads the run used.
    """
    want = np.uint8 if in_dtype == IN_FP8_E4M3 else np.uint16
    q = np.ascontiguousarray(q)
    k = np.ascontiguousarray(k)
    v = np.ascontiguousarray(v)
    if q.dtype != want or k.dtype != want or v.dtype != want:
        raise TypeError(f"storage arrays must be {want}")
    B, Sq, Hq, D = q.shape
    _, Sk, Hkv, _ = k.shape
    if rows is not None:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int32)
        nrows, rows_ptr = rows_arr.size, rows_arr.ctypes.data
    else:
        rows_arr, nrows, rows_ptr = None, Sq, None
    O = np.empty((B, Hq, nrows, D), dtype=np.float64)
    LSE = np.empty((B, Hq, nrows), dtype=np.float64)
    widen_o = np.zeros((B, Hq, nrows), dtype=np.float64)
    widen_lse = np.zeros((B, Hq, nrows), dtype=np.float64)
    nflag = np.zeros((B, Hq, nrows), dtype=np.int32)
    rc = lib().oracle_attn(q.ctypes.data, k.ctypes.data, v.ctypes.data, in_dtype, B, Hq, Hkv, Sq,
                           Sk, D, int(bool(causal)), softmax_scale, q_descale, k_descale,
                           v_descale, mode, tile_n, kv_order, float(tau), kmax, int(drop_tail), p_round,
                           p_off,
                           float(tie_eps), rows_ptr, nrows, O.ctypes.data, LSE.ctypes.data,
                           widen_o.ctypes.data, widen_lse.ctypes.data, nflag.ctypes.data, nthreads)
    if rc < 0:
        raise ValueError(f"oracle_attn failed: {rc}")
    return {"O": O, "LSE": LSE, "widen_o": widen_o, "widen_lse": widen_lse, "nflag": nflag,
            "threads": rc}
