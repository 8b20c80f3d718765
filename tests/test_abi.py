"""The C-ABI library loads and exports every symbol that include/attn.h declares (no GPU needed)."""
import ctypes
import re
from pathlib import Path

from paper_2609_33586_b200 import binding, build

ROOT = Path(__file__).resolve().parent.parent


def _declared_functions():
    text = (ROOT / "include" / "attn.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(attn_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    lib_path = build.build()
    L = ctypes.CDLL(str(lib_path))
    declared = _declared_functions()
    assert set(declared) == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_host_only_entry_points_work_without_a_gpu():
    assert binding.version().startswith("rowmax-attn-b200")
    assert binding.status_string(0) == "ok" and "shape" in binding.status_string(-2)
    for in_dtype, mode, fmt, off in ((0, 2, binding.P_BF16, 0), (1, 0, binding.P_E4M3, 8), (1, 2, binding.P_E5M2, 15),
                                     (1, 3, binding.P_E5M2, 15), (1, 4, binding.P_E4M3, 8), (1, 5, binding.P_E4M3, 8)):
        s = binding.get_schedule(128, in_dtype, mode, True)
        assert (s["tile_m"], s["tile_n"], s["kv_order"], s["rescale_tau"], s["pot_kmax"]) == (128, 128, 1, 0.0, 20)
        assert (s["p_format"], s["p_offset_log2"]) == (fmt, off)
    assert binding.lib().attn_get_schedule(96, 0, 0, 0, *([None] * 7)) == -2
    # argument validation happens before any CUDA call
    assert binding.attn_fwd_raw(None, None, None, None, None, 1, 1, 1, 1, 1, 64, 0, 1.0, 0, 0, 1, 1, 1, None) == -1
    assert binding.lib().attn_weight_map(None, None, 0, 2, None) == 0
    assert binding.lib().attn_weight_map(None, None, 4, 2, None) == -1
