"""Thin ctypes binding over the C-ABI library declared in ``include/attn.h``.

Argument marshalling only: every step of the attention forward runs in the CUDA kernels of
``libattn_b200.so``.  There is no fallback: if the library is missing or fails to load, importing a
function from here raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

W_EXACT, W_POT, W_H15, W_H15K2, W_H15K3, W_EXACT_POLY = 0, 1, 2, 3, 4, 5
IN_BF16, IN_FP8_E4M3, IN_FP16 = 0, 1, 2
P_BF16, P_E4M3, P_E5M2, P_FP16 = 0, 1, 2, 3
MODES = {"exact": W_EXACT, "pot": W_POT, "h15": W_H15, "h15k2": W_H15K2, "h15k3": W_H15K3,
         "exact_poly": W_EXACT_POLY}

_LIB_PATH = Path(__file__).resolve().parent / "libattn_b200.so"
_lib = None

EXPORTS = ("attn_fwd", "attn_fwd_tau", "attn_fwd_pot", "attn_fwd_exact_emulated", "attn_weight_map", "attn_weight_map_pot", "attn_weight_map_fused", "attn_get_schedule", "attn_device_status",
           "attn_device_status_code", "attn_selftest_wait", "attn_device_status_reset", "attn_launch_count", "attn_status_string",
           "attn_last_cuda_error", "attn_version")


class AttnError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what} failed: {code} ({status_string(code)})")
        self.code = code


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2609_33586_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(str(_LIB_PATH))
        vp, i, f = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
        L.attn_fwd.restype = i
        L.attn_fwd.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, i, f, f, f, vp]
        L.attn_fwd_tau.restype = i
        L.attn_fwd_tau.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, i, f, f, f, f, vp]
        L.attn_fwd_pot.restype = i
        L.attn_fwd_pot.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, f, f, f, i, i, vp]
        L.attn_fwd_exact_emulated.restype = i
        L.attn_fwd_exact_emulated.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, f, f, f, i, vp]
        L.attn_weight_map.restype = i
        L.attn_weight_map.argtypes = [vp, vp, ctypes.c_size_t, i, vp]
        L.attn_weight_map_pot.restype = i
        L.attn_weight_map_pot.argtypes = [vp, vp, ctypes.c_size_t, i, i, vp]
        L.attn_weight_map_fused.restype = i
        L.attn_weight_map_fused.argtypes = [vp, vp, ctypes.c_size_t, i, i, i, i, vp]
        L.attn_get_schedule.restype = i
        L.attn_get_schedule.argtypes = [i, i, i, i] + [vp] * 7
        L.attn_device_status.restype = i
        L.attn_device_status_code.restype = i
        L.attn_selftest_wait.restype = i
        L.attn_selftest_wait.argtypes = [ctypes.c_longlong, vp]
        L.attn_device_status_reset.restype = i
        L.attn_launch_count.restype = ctypes.c_ulonglong
        L.attn_status_string.restype = ctypes.c_char_p
        L.attn_status_string.argtypes = [i]
        L.attn_last_cuda_error.restype = i
        L.attn_version.restype = ctypes.c_char_p
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().attn_status_string(int(code)).decode()


def version() -> str:
    return lib().attn_version().decode()


def launch_count() -> int:
    return int(lib().attn_launch_count())


def device_status() -> int:
    return int(lib().attn_device_status())


def device_status_code() -> int:
    """The raw status word: 0, or role << 8 | barrier id of the first wait that ran out."""
    return int(lib().attn_device_status_code())


def selftest_wait(limit_cycles: int, stream=None) -> None:
    """Launches the one-warp kernel whose bounded wait runs out (sets the sticky status word)."""
    rc = lib().attn_selftest_wait(int(limit_cycles), _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_selftest_wait")


def device_status_reset() -> None:
    rc = lib().attn_device_status_reset()
    if rc != 0:
        raise AttnError(rc, "attn_device_status_reset")


def get_schedule(D: int, in_dtype: int, weight_mode: int, causal: bool) -> dict:
    ints = [ctypes.c_int() for _ in range(6)]
    tau = ctypes.c_float()
    rc = lib().attn_get_schedule(D, in_dtype, weight_mode, int(causal), ctypes.addressof(ints[0]),
                                 ctypes.addressof(ints[1]), ctypes.addressof(ints[2]),
                                 ctypes.addressof(tau), ctypes.addressof(ints[3]),
                                 ctypes.addressof(ints[4]), ctypes.addressof(ints[5]))
    if rc != 0:
        raise AttnError(rc, "attn_get_schedule")
    return {"tile_m": ints[0].value, "tile_n": ints[1].value, "kv_order": ints[2].value,
            "rescale_tau": tau.value, "pot_kmax": ints[3].value, "p_format": ints[4].value,
            "p_offset_log2": ints[5].value}


def _stream_ptr(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def in_dtype_of(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return IN_BF16
    if t.dtype == torch.float8_e4m3fn:
        return IN_FP8_E4M3
    if t.dtype == torch.float16:
        return IN_FP16
    raise TypeError(f"unsupported storage dtype {t.dtype}")


def attn_fwd_raw(q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, B, Hq, Hkv, Sq, Sk, D, causal, softmax_scale,
                 weight_mode, in_dtype, q_descale, k_descale, v_descale, stream_ptr, rescale_tau=None,
                 pot_tail=None, poly_eighths=None) -> int:
    """Direct call with integer device addresses; returns the status code.  With `rescale_tau` the
    call goes to attn_fwd_tau, with `pot_tail` = (K_max, drop_tail) to attn_fwd_pot, with `poly_eighths`
    to attn_fwd_exact_emulated."""
    if poly_eighths is not None:
        return lib().attn_fwd_exact_emulated(q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, B, Hq, Hkv, Sq, Sk, D, int(causal),
                                             softmax_scale, in_dtype, q_descale, k_descale, v_descale,
                                             int(poly_eighths), stream_ptr)
    if pot_tail is not None:
        return lib().attn_fwd_pot(q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, B, Hq, Hkv, Sq, Sk, D, int(causal),
                                  softmax_scale, in_dtype, q_descale, k_descale, v_descale,
                                  int(pot_tail[0]), int(bool(pot_tail[1])), stream_ptr)
    if rescale_tau is None:
        return lib().attn_fwd(q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, B, Hq, Hkv, Sq, Sk, D, int(causal),
                              softmax_scale, weight_mode, in_dtype, q_descale, k_descale, v_descale,
                              stream_ptr)
    return lib().attn_fwd_tau(q_ptr, k_ptr, v_ptr, o_ptr, lse_ptr, B, Hq, Hkv, Sq, Sk, D, int(causal),
                              softmax_scale, weight_mode, in_dtype, q_descale, k_descale, v_descale,
                              rescale_tau, stream_ptr)


def attn_fwd(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, *, causal: bool, softmax_scale: float,
             weight_mode: int, q_descale: float = 1.0, k_descale: float = 1.0, v_descale: float = 1.0,
             out: torch.Tensor | None = None, lse: torch.Tensor | None = None, return_lse: bool = True,
             rescale_tau: float | None = None, pot_tail=None, poly_eighths=None, stream=None):
    """q (B,Sq,Hq,D), k/v (B,Sk,Hkv,D): contiguous CUDA tensors, bf16, float16 or float8_e4m3fn.
    Returns (O bf16 (B,Sq,Hq,D), LSE fp32 (B,Hq,Sq) or None).  `rescale_tau` (bf16 inputs only) selects
    the deferred-rescale entry point attn_fwd_tau; `pot_tail` = (K_max, drop_tail) selects attn_fwd_pot
    (Rowmax-PoT with that tail; `weight_mode` must then be W_POT); `poly_eighths` (1..4) selects
    attn_fwd_exact_emulated (`weight_mode` must then be W_EXACT_POLY)."""
    if poly_eighths is not None and weight_mode != W_EXACT_POLY:
        raise ValueError("poly_eighths goes with weight_mode = W_EXACT_POLY")
    if pot_tail is not None and weight_mode != W_POT:
        raise ValueError("pot_tail goes with weight_mode = W_POT")
    for t in (q, k, v):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("q, k, v must be contiguous CUDA tensors")
    dt = in_dtype_of(q)
    if in_dtype_of(k) != dt or in_dtype_of(v) != dt:
        raise TypeError("q, k, v must share one storage dtype")
    B, Sq, Hq, D = q.shape
    Bk, Sk, Hkv, Dk = k.shape
    if v.shape != k.shape or Bk != B or Dk != D:
        raise ValueError("shape mismatch between q, k, v")
    if out is None:
        out = torch.empty((B, Sq, Hq, D), dtype=torch.bfloat16, device=q.device)
    if lse is None and return_lse:
        lse = torch.empty((B, Hq, Sq), dtype=torch.float32, device=q.device)
    rc = attn_fwd_raw(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                      lse.data_ptr() if lse is not None else None, B, Hq, Hkv, Sq, Sk, D, causal,
                      softmax_scale, weight_mode, dt, q_descale, k_descale, v_descale,
                      _stream_ptr(stream), rescale_tau, pot_tail, poly_eighths)
    if rc != 0:
        raise AttnError(rc, "attn_fwd")
    return out, lse


def weight_map(x: torch.Tensor, weight_mode: int, out: torch.Tensor | None = None, stream=None):
    """Applies the device weight map to a contiguous fp32 CUDA tensor of base-two offsets."""
    if not x.is_cuda or x.dtype != torch.float32 or not x.is_contiguous():
        raise ValueError("x must be a contiguous fp32 CUDA tensor")
    if out is None:
        out = torch.empty_like(x)
    rc = lib().attn_weight_map(x.data_ptr(), out.data_ptr(), x.numel(), weight_mode, _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_weight_map")
    return out


def weight_map_pot(x: torch.Tensor, kmax: int, drop_tail: bool, out: torch.Tensor | None = None, stream=None):
    """Rowmax-PoT with the tail index `kmax`, clamped or dropped, on a contiguous fp32 CUDA tensor of offsets."""
    if not x.is_cuda or x.dtype != torch.float32 or not x.is_contiguous():
        raise ValueError("x must be a contiguous fp32 CUDA tensor")
    if out is None:
        out = torch.empty_like(x)
    rc = lib().attn_weight_map_pot(x.data_ptr(), out.data_ptr(), x.numel(), int(kmax), int(bool(drop_tail)), _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_weight_map_pot")
    return out


def weight_map_fused(x: torch.Tensor, weight_mode: int, in_dtype: int, kmax: int = 20, drop_tail: bool = False,
                     out: torch.Tensor | None = None, stream=None):
    """The weights as the fused kernel's hot loop stores them in P for inputs of storage type `in_dtype`."""
    if not x.is_cuda or x.dtype != torch.float32 or not x.is_contiguous():
        raise ValueError("x must be a contiguous fp32 CUDA tensor")
    if out is None:
        out = torch.empty_like(x)
    rc = lib().attn_weight_map_fused(x.data_ptr(), out.data_ptr(), x.numel(), weight_mode, in_dtype, int(kmax),
                                     int(bool(drop_tail)), _stream_ptr(stream))
    if rc != 0:
        raise AttnError(rc, "attn_weight_map_fused")
    return out
