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
    # a masked score (-inf) and anything below -127 weigh exactly nothing, as with the hardware ex2
    assert _gpu_map(np.array([-np.inf, -127.0, -200.0], np.float32), binding.W_EXACT_POLY).tolist() == [0.0, 0.0, 0.0]


def test_in_place_and_empty():
    x = torch.tensor([-1.5, 0.0], device="cuda")
    binding.weight_map(x, orc.W_H15, out=x)
    assert x.cpu().tolist() == [0.375, 1.0]
    e = torch.empty(0, device="cuda")
    assert binding.weight_map(e, orc.W_H15).numel() == 0


@pytest.mark.parametrize("drop", [False, True])
@pytest.mark.parametrize("kmax", [1, 8, 12, 20, 48, 125])
def test_pot_tail_map_is_bit_exact_on_the_sweep(kmax, drop):
    for x in (inputs.weight_map_sweep(), inputs.paper_bit_test_set()):
        x = x[x <= 0.5]
        got = binding.weight_map_pot(torch.from_numpy(x).cuda(), kmax, drop).cpu().numpy()
        want = orc.weight_map(x, orc.W_POT, kmax=kmax, drop_tail=drop).astype(np.float32)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def _chunks_of(x, pred):
    """Offsets arranged so that chunks of 32 are uniform in `pred` (the fused loop picks its variant per chunk)."""
    a, b = x[pred], x[~pred]
    pad = (-len(a)) % 32
    return np.concatenate([a, np.zeros(pad, np.float32), b]).astype(np.float32)


# storage type -> (lowest offset whose weight P still holds exactly, per mode)
_P_FLOOR = {
    binding.IN_BF16: {orc.W_H15: -126.0, orc.W_H15K2: -126.0, orc.W_H15K3: -126.0, orc.W_POT: -126.0},
    binding.IN_FP16: {orc.W_H15: -23.0, orc.W_POT: -24.0},     # fp16 subnormals: 1.5 * 2^k needs k >= -23
    binding.IN_FP8_E4M3: {orc.W_H15: -29.0, orc.W_H15K2: -29.0, orc.W_H15K3: -14.0, orc.W_POT: -29.0},
}


@pytest.mark.parametrize("in_dtype", [binding.IN_BF16, binding.IN_FP16, binding.IN_FP8_E4M3])
@pytest.mark.parametrize("mode", [orc.W_H15, orc.W_H15K2, orc.W_H15K3, orc.W_POT])
def test_fused_loop_instantiations_are_bit_exact_where_p_holds_the_weight(mode, in_dtype):
    # the instantiations attn_fwd runs (h15 family without the per-score clamp, P offset folded into the weight,
    # pot on the negated offset), read back from the packed P words
    if mode not in _P_FLOOR[in_dtype]:
        pytest.skip("not built for this storage type")
    floor = _P_FLOOR[in_dtype][mode]
    kmax = {binding.IN_BF16: 20, binding.IN_FP16: 20, binding.IN_FP8_E4M3: 20}[in_dtype]
    for x in (inputs.weight_map_sweep(), inputs.paper_bit_test_set()):
        x = x[np.isfinite(x) & (x <= 0.0)]
        x = _chunks_of(x, x >= -125.0)                    # chunks entirely above -125 take the unclamped variant
        got = binding.weight_map_fused(torch.from_numpy(x).cuda(), mode, in_dtype, kmax).cpu().numpy()
        want = orc.weight_map(x, mode, kmax=kmax).astype(np.float32)
        held = x >= floor
        if mode == orc.W_POT:       # ties: see test_fused_loop_pot_tail
            held = held & ~((x * 2 == np.floor(x * 2)) & (x != np.floor(x)))
        k = {orc.W_H15: 1, orc.W_H15K2: 2, orc.W_H15K3: 3}.get(mode, 0)
        if k > 0 and in_dtype != binding.IN_FP8_E4M3:
            # the saturating form of the 16-bit paths may decide a tie, or an offset within 2^-20 (relative) of one,
            # either way; anywhere else it is bit-exact (see attn_weight_map_fused in attn.h)
            u = x.astype(np.float64) * 2.0 ** k
            dist = np.abs(u - (np.floor(u) + 0.5))
            near = dist < 2.0 ** -20 * np.maximum(1.0, np.abs(u))
            lo = orc.weight_map(np.nextafter(x, np.float32(-np.inf)) - np.float32(2.0 ** -18) * np.abs(x), mode).astype(np.float32)
            hi = orc.weight_map(np.minimum(np.nextafter(x, np.float32(np.inf)) + np.float32(2.0 ** -18) * np.abs(x), np.float32(0)), mode).astype(np.float32)
            ok_near = (got == lo) | (got == hi) | (got == want)
            assert np.all(ok_near[held & near]) and near.sum() > 100
            held = held & ~near
        assert np.array_equal(got[held].view(np.uint32), want[held].view(np.uint32))
        # below that P rounds in its subnormal range and then underflows to zero: never more than one binade off
        assert np.all(got[~held] >= 0) and np.all(got[~held] <= want[~held] * 2.0 + 2.0 ** -120)


@pytest.mark.parametrize("in_dtype,kmax", [(binding.IN_BF16, 8), (binding.IN_BF16, 48), (binding.IN_FP8_E4M3, 12), (binding.IN_FP8_E4M3, 29),
                                           (binding.IN_FP16, 12)])
@pytest.mark.parametrize("drop", [False, True])
def test_fused_loop_pot_tail(in_dtype, kmax, drop):
    x = inputs.weight_map_sweep()
    x = x[np.isfinite(x) & (x <= 0.0)]
    got = binding.weight_map_fused(torch.from_numpy(x).cuda(), orc.W_POT, in_dtype, kmax, drop).cpu().numpy()
    want = orc.weight_map(x, orc.W_POT, kmax=kmax, drop_tail=drop).astype(np.float32)
    # the fused loop rounds the offset to nearest-even where the definition sends ties down: equal everywhere but at
    # an exact tie x = -(d + 1/2), where either neighbour may come out (the boundary of a dropped tail is kept exact)
    tie = (x * 2 == np.floor(x * 2)) & (x != np.floor(x)) & (x > -(kmax + 0.5))
    assert np.array_equal(got[~tie].view(np.uint32), want[~tie].view(np.uint32))
    assert np.all((got[tie] == want[tie]) | (got[tie] == 2 * want[tie])) and tie.sum() >= kmax - 1


@pytest.mark.parametrize("in_dtype,rel", [(binding.IN_BF16, 2.0 ** -8), (binding.IN_FP16, 2.0 ** -11), (binding.IN_FP8_E4M3, 2.0 ** -4)])
def test_fused_loop_exact_mode_is_the_exponential_rounded_to_the_format_of_p(in_dtype, rel):
    x = np.linspace(-7.5, 0.0, 4096, dtype=np.float32)
    got = binding.weight_map_fused(torch.from_numpy(x).cuda(), orc.W_EXACT, in_dtype).cpu().numpy().astype(np.float64)
    want = orc.weight_map(x, orc.W_EXACT)
    assert np.max(np.abs(got / want - 1.0)) <= rel * 1.01
