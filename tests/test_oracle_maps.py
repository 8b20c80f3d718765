"""Pins for the CPU oracle's weight maps and storage decoders (no GPU).

Each test ties the oracle to something other than itself: values the paper prints, closed forms,
invariants, an independent coding of the same definition, or a library routine.
"""
import math

import numpy as np
import pytest
import torch

from oracle import cpu_oracle as orc
from paper_2609_33586_b200 import inputs

LOG2_1P5 = math.log2(1.5)


def _read_points(path):
    pts = []
    for line in path.read_text().splitlines():
        line = line.split("#")[0].strip()
        if line:
            a = line.split()
            pts.append((float(a[0]), float(a[1])))
    return pts


# ---- values printed by the paper ----------------------------------------------------------------

def test_h15_golden_points(golden_dir):
    for x, want in _read_points(golden_dir / "h15_points.txt"):
        got = orc.weight_map(np.array([x], np.float32), orc.W_H15)[0]
        assert got == want, (x, got, want)


def test_pot_golden_points(golden_dir):
    for x, want in _read_points(golden_dir / "pot_points.txt"):
        got = orc.weight_map(np.array([x], np.float32), orc.W_POT)[0]
        assert got == want, (x, got, want)


def test_h15_envelope_and_spacing(golden_dir):
    g = dict(l.split() for l in (golden_dir / "h15_envelope.txt").read_text().splitlines()
             if l and not l.startswith("#"))
    assert float(g["lower"]) == -0.25
    assert abs(float(g["upper"]) - (LOG2_1P5 - 0.25)) < 5e-6
    x = inputs.paper_bit_test_set()
    w = orc.weight_map(x, orc.W_H15)
    eps = np.log2(w) - x.astype(np.float64)
    assert eps.min() >= -0.25 and eps.max() <= LOG2_1P5 - 0.25
    # both endpoints are approached: the envelope is tight, not merely valid
    assert eps.min() < -0.2499 and eps.max() > LOG2_1P5 - 0.2501
    vals = np.unique(np.log2(w))
    gaps = np.unique(np.round(np.diff(vals), 12))
    assert len(gaps) == 2
    assert abs(gaps[1] - LOG2_1P5) < 1e-9 and abs(gaps[0] - (1 - LOG2_1P5)) < 1e-9
    assert abs(gaps[1] - float(g["spacing_a"])) < 5e-4 and abs(gaps[0] - float(g["spacing_b"])) < 5e-4


# ---- structural invariants ----------------------------------------------------------------------

def test_h15_range_is_one_or_one_and_a_half_times_power_of_two():
    x = inputs.weight_map_sweep()
    w = orc.weight_map(x, orc.W_H15)
    mant, _ = np.frexp(w)  # w = mant * 2^e, mant in [0.5, 1)
    assert set(np.unique(mant)) <= {0.5, 0.75}


def test_maps_are_monotone_and_one_at_anchor():
    x = np.sort(inputs.weight_map_sweep())
    for mode in (orc.W_EXACT, orc.W_POT, orc.W_H15):
        w = orc.weight_map(x, mode)
        assert np.all(np.diff(w) >= 0), mode
        assert orc.weight_map(np.array([0.0, -0.0], np.float32), mode).tolist() == [1.0, 1.0]


def test_h15_octave_equivariance():
    rng = np.random.default_rng(1)
    x = rng.uniform(-60, 0, 20000).astype(np.float32)
    x = (np.round(x * 4096) / 4096).astype(np.float32)  # exact under integer shifts
    base = orc.weight_map(x, orc.W_H15)
    for j in (-7, -1, 1, 3):
        shifted = orc.weight_map((x + np.float32(j)).astype(np.float32), orc.W_H15)
        assert np.array_equal(shifted, base * 2.0 ** j)


def test_h15_equals_schraudolph_on_half_integer_rounded_input():
    # H(x) = S(Q_1/2(x)) with S(x) = 2^floor(x) (1 + x - floor(x)), written out independently here.
    x = inputs.paper_bit_test_set()
    q = np.rint(2.0 * x.astype(np.float64)) / 2.0  # np.rint rounds half to even
    s = np.exp2(np.floor(q)) * (1.0 + q - np.floor(q))
    assert np.array_equal(orc.weight_map(x, orc.W_H15), s)


def _h15_add_and_shift(x32):
    """The construction of App. B.1 "Implementation", in NumPy fp32/int32 arithmetic: clamp the
    doubled input at -252, add 0x4B400000 as a float (round to nearest even), shift the bit
    pattern left by 22 and add the bit pattern of 1.0."""
    two_x = np.maximum(x32 * np.float32(2.0), np.float32(-252.0)).astype(np.float32)
    magic = np.array([0x4B400000], dtype=np.uint32).view(np.float32)[0]
    t = (two_x + magic).astype(np.float32)
    bits = t.view(np.uint32)
    out = (bits << np.uint32(22)) + np.uint32(0x3F800000)
    return out.view(np.float32)


def test_h15_equals_add_and_shift_bit_construction():
    for x in (inputs.paper_bit_test_set(), inputs.weight_map_sweep()):
        x = x[np.isfinite(x) & (x > -1e6) & (x < 127)]
        want = _h15_add_and_shift(x)
        got = orc.weight_map(x, orc.W_H15).astype(np.float32)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


# ---- the family H15 belongs to: S(Q_{2^-k}(x)), k = 2, 3 (App. B "Exponential-map ablation") ----

def _schraudolph(q):
    return np.exp2(np.floor(q)) * (1.0 + q - np.floor(q))


@pytest.mark.parametrize("k,mode", [(2, orc.W_H15K2), (3, orc.W_H15K3)])
def test_h15_family_equals_schraudolph_on_rounded_input_and_the_shift_construction(k, mode):
    x = inputs.paper_bit_test_set()
    q = np.rint(x.astype(np.float64) * 2 ** k) / 2 ** k           # independent coding of Q_{2^-k}
    got = orc.weight_map(x, mode)
    assert np.array_equal(got, _schraudolph(q))
    # the add-and-shift pattern with 2^k x and a left shift by 23 - k
    magic = np.array([0x4B400000], dtype=np.uint32).view(np.float32)[0]
    t = (np.maximum(x * np.float32(2 ** k), np.float32(-126 * 2 ** k)).astype(np.float32) + magic).astype(np.float32)
    bits = (t.view(np.uint32) << np.uint32(23 - k)) + np.uint32(0x3F800000)
    assert np.array_equal(got.astype(np.float32).view(np.uint32), bits)


def test_h15_family_k1_is_h15_and_envelopes_shrink_with_k():
    x = inputs.paper_bit_test_set()
    assert np.array_equal(orc.weight_map(x, orc.W_H15), _schraudolph(np.rint(2.0 * x.astype(np.float64)) / 2.0))
    interp = 0.08607133205593432       # max of log2(1 + f) - f, attained at f = 1/ln 2 - 1
    for k, mode in ((2, orc.W_H15K2), (3, orc.W_H15K3)):
        w = orc.weight_map(x, mode)
        eps = np.log2(w) - x.astype(np.float64)
        half_step = 2.0 ** -(k + 1)   # |q - x| <= half an input step; log2 S(q) - q lies in [0, interp]
        assert eps.min() >= -half_step - 1e-12 and eps.max() <= interp + half_step + 1e-12
        xs = np.sort(inputs.weight_map_sweep())
        ws = orc.weight_map(xs, mode)
        assert np.all(np.diff(ws) >= 0)
        assert orc.weight_map(np.array([0.0, -126.0, -200.0, -np.inf], np.float32), mode).tolist() == \
            [1.0, 2.0 ** -126, 2.0 ** -126, 2.0 ** -126]
        frac_bits = np.unique(np.frexp(w)[0] * 2 ** (k + 1))       # mantissa in [0.5,1) has k fraction bits
        assert np.all(frac_bits == np.round(frac_bits))


def test_h15_minus_infinity_is_the_clamp_value():
    w = orc.weight_map(np.array([-np.inf, -150.0, -126.0], np.float32), orc.W_H15)
    assert np.all(w == 2.0 ** -126)
    assert np.array(w, np.float32).view(np.uint32).tolist() == [0x00800000] * 3


def test_pot_properties():
    x = inputs.weight_map_sweep()
    x = x[np.isfinite(x) & (x <= 0)]
    w = orc.weight_map(x, orc.W_POT)
    d = -np.log2(w)
    assert np.array_equal(d, np.round(d)) and d.min() == 0 and d.max() == 20
    body = x >= -20.5
    assert np.all(np.abs(np.log2(w[body]) - x[body]) <= 0.5)  # |eps| <= ln2/2 in octaves, m = 1
    # K_max is a parameter: the tail floors at 2^-K_max
    assert orc.weight_map(np.array([-50.0], np.float32), orc.W_POT, kmax=8)[0] == 2.0 ** -8
    # brute force on the definition with exact rationals (all x here are multiples of 2^-10)
    from fractions import Fraction
    for xv in x[::997]:
        y = -Fraction(float(xv))
        dd = min(20, math.floor(y + Fraction(1, 2)))
        assert orc.weight_map(np.array([xv], np.float32), orc.W_POT)[0] == 2.0 ** -dd


@pytest.mark.parametrize("kmax", [8, 12, 20, 48])
def test_pot_tail_clamp_and_drop(kmax):
    # App. A, after Eq. rowmax-pot: the main point clamps the tail at K_max (full support); the tail-drop
    # variant removes the keys whose index exceeds K_max.  Index d = floor(y + 1/2), y = -x.
    x = inputs.weight_map_sweep()
    x = x[np.isfinite(x) & (x <= 0)]
    clamp = orc.weight_map(x, orc.W_POT, kmax=kmax)
    drop = orc.weight_map(x, orc.W_POT, kmax=kmax, drop_tail=True)
    d = np.floor(-x.astype(np.float64) + 0.5)
    assert np.array_equal(clamp, 2.0 ** -np.minimum(d, kmax))
    assert np.array_equal(drop, np.where(d > kmax, 0.0, 2.0 ** -d))
    assert np.array_equal(clamp[d <= kmax], drop[d <= kmax])            # the two agree on the body
    one = lambda v, **kw: orc.weight_map(np.array([v], np.float32), orc.W_POT, kmax=kmax, **kw)[0]   # noqa: E731
    assert one(-(kmax + 1)) == 2.0 ** -kmax and one(-(kmax + 1), drop_tail=True) == 0.0
    assert one(-kmax) == 2.0 ** -kmax == one(-kmax, drop_tail=True)
    assert one(-(kmax + 0.5), drop_tail=True) == 0.0                     # ties go up in d: d = K_max + 1 is dropped
    assert one(np.nextafter(np.float32(-(kmax + 0.5)), np.float32(0)), drop_tail=True) == 2.0 ** -kmax
    assert one(-np.inf) == 2.0 ** -kmax and one(-np.inf, drop_tail=True) == 0.0
    order = np.argsort(x, kind="stable")
    assert np.all(np.diff(clamp[order]) >= 0) and np.all(np.diff(drop[order]) >= 0)   # both monotone
    assert one(0.0) == 1.0 == one(0.0, drop_tail=True)


def test_pot_no_double_rounding_at_fp32_edge():
    # y = 0.5 - 2^-25 is an fp32 value; y + 0.5 rounds to 1.0 in fp32 but floor(y + 1/2) is 0.
    x = np.float32(-(0.5 - 2.0 ** -25))
    assert float(x) != -0.5
    assert orc.weight_map(np.array([x]), orc.W_POT)[0] == 1.0


def test_exact_map_is_exp2():
    x = inputs.weight_map_sweep()
    x = x[np.isfinite(x)]
    w = orc.weight_map(x, orc.W_EXACT)
    assert np.allclose(w, np.exp2(x.astype(np.float64)), rtol=1e-15, atol=0)
    assert orc.weight_map(np.array([-np.inf], np.float32), orc.W_EXACT)[0] == 0.0
    # natural-exponential form of Eq. m-exact: exp(-Delta) with Delta = -x ln 2
    assert np.allclose(w, np.exp(x.astype(np.float64) * math.log(2.0)), rtol=1e-13, atol=0)


# ---- storage decoders against the library casts ------------------------------------------------

def test_bf16_decoder_matches_torch_for_every_pattern():
    bits = np.arange(65536, dtype=np.uint16)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([orc.decode_bf16(int(b)) for b in bits])
    both_nan = np.isnan(ref) & np.isnan(got)
    assert np.all((ref == got) | both_nan)
    assert np.array_equal(np.signbit(ref[~both_nan]), np.signbit(got[~both_nan]))


def test_fp16_decoder_matches_torch_for_every_pattern():
    bits = np.arange(65536, dtype=np.uint16)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.float16).to(torch.float64).numpy()
    got = np.array([orc.decode_fp16(int(b)) for b in bits])
    both_nan = np.isnan(ref) & np.isnan(got)
    assert np.all((ref == got) | both_nan)
    assert np.array_equal(np.signbit(ref[~both_nan]), np.signbit(got[~both_nan]))
    assert got[0x7BFF] == 65504.0 and got[0x0001] == 2.0 ** -24


def test_e4m3_decoder_matches_torch_for_every_pattern():
    bits = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(bits).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = np.array([orc.decode_e4m3(int(b)) for b in bits])
    both_nan = np.isnan(ref) & np.isnan(got)
    assert np.all((ref == got) | both_nan)
    assert got[0x7E] == 448.0 and np.isnan(got[0x7F])


def test_bad_mode_is_rejected():
    with pytest.raises(ValueError):
        orc.weight_map(np.zeros(1, np.float32), 7)
