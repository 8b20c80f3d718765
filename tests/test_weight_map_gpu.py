"""GPU gate for the device weight maps: bit-exact against the CPU oracle on a dense sweep of fp32
offsets (includes every rounding tie, 0, values below the clamp and -inf)."""
import numpy as np
import pytest
import torch

from oracle import cpu_oracle as orc
from paper_2609_33586_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _gpu_map(x, mode):
    xt = torch.from_numpy(x).cuda()
    return binding.weight_map(xt, mode).cpu().numpy()


@pytest.mark.parametrize("mode", [orc.W_H15, orc.W_POT, orc.W_H15K2, orc.W_H15K3])
def test_rounding_maps_are_bit_exact_on_the_sweep(mode):
    for x in (inputs.weight_map_sweep(), inputs.paper_bit_test_set()):
        if mode == orc.W_POT:
            x = x[x <= 0.5]          # the product only defines pot at or below the anchor (+ rounding residue)
        got = _gpu_map(x, mode)
        want = orc.weight_map(x, mode).astype(np.float32)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_h15_special_points():
    x = np.array([0.0, -0.0, -1.5, -126.0, -150.0, -np.inf, 0.75, 1.5], np.float32)
    got = _gpu_map(x, orc.W_H15)
    assert got.tolist() == [1.0, 1.0, 0.375, 2.0 ** -126, 2.0 ** -126, 2.0 ** -126, 2.0, 3.0]
    assert got.view(np.uint32)[5] == 0x00800000


def test_exact_map_within_two_ulp_and_flushes_subnormals():
    x = inputs.weight_map_sweep()
    x = x[np.isfinite(x)]
    got = _gpu_map(x, orc.W_EXACT).astype(np.float64)
    want = orc.weight_map(x, orc.W_EXACT)
    normal = want >= 2.0 ** -126
    rel = np.abs(got[normal] - want[normal]) / want[normal]
    assert rel.max() <= 2 * 2.0 ** -23 + 2.0 ** -22 * 0  # ex2.approx: 2 ulp
    assert np.all(got[~normal] <= 2.0 ** -126)             # flushed (or the smallest normal)
    assert _gpu_map(np.array([-np.inf], np.float32), orc.W_EXACT)[0] == 0.0


def test_emulated_exact_map_is_within_its_stated_error():
    x = inputs.weight_map_sweep()
    x = x[np.isfinite(x) & (x >= -126.0)]
    got = _gpu_map(x, binding.W_EXACT_POLY).astype(np.float64)
    want = orc.weight_map(x, orc.W_EXACT)
    assert np.max(np.abs(got / want - 1.0)) <= 1.1e-4
    assert np.all(np.diff(got[np.argsort(x, kind="stable")]) >= 0)          # monotone, continuous across octaves
    ints = np.arange(-126, 17, dtype=np.float32)
    assert np.array_equal(_gpu_map(ints, binding.W_EXACT_POLY), np.exp2(ints.astype(np.float64)).astype(np.float32))


def test_in_place_and_empty():
    x = torch.tensor([-1.5, 0.0], device="cuda")
    binding.weight_map(x, orc.W_H15, out=x)
    assert x.cpu().tolist() == [0.375, 1.0]
    e = torch.empty(0, device="cuda")
    assert binding.weight_map(e, orc.W_H15).numel() == 0
