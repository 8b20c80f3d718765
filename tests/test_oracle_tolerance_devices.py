"""Pins for the two devices of this build that the parity comparison leans on and that have no
counterpart in the paper (no GPU needed):

  - the P-storage diagnostic (`p_round`): rounding of a weight to bfloat16, e4m3 or e5m2, pinned
    against a library's casts on dense sweeps that contain every tie, the subnormal range and the
    saturation point;
  - the tie-widening bound: a score that sits on a rounding boundary of the weight map may land on
    either side in fp32; the oracle returns a bound on what such flips can do to O and LSE.  Here every
    flagged score (and random subsets of them) is moved across its boundary and the change is checked
    against the bound, so the bound is a proved property, not a fitted tolerance.
"""
import math

import numpy as np
import pytest
import torch

from oracle import cpu_oracle as orc
from paper_2609_33586_b200.inputs import storage_bits

from test_oracle_attention import _bf16_bits, _numpy_online

LOG2E = 1.4426950408889634


# ---- p_round against library casts -------------------------------------------------------------

def _sweep(frac_bits, e_lo, e_hi):
    """Every positive value with `frac_bits` + 2 fraction bits for exponents e_lo..e_hi (contains all
    representable values of the target format, every midpoint between neighbours and the quarter
    points), each with its two float64 neighbours a hair below and above."""
    m = 1.0 + np.arange(0, 2 ** (frac_bits + 2)) / 2.0 ** (frac_bits + 2)
    v = np.concatenate([m * 2.0 ** e for e in range(e_lo, e_hi + 1)])
    return np.concatenate([v, v * (1 - 2.0 ** -30), v * (1 + 2.0 ** -30)])


def _torch_cast(v, dtype, vmax):
    t = torch.from_numpy(np.minimum(v, vmax)).to(torch.float32)      # the diagnostic saturates; torch does not
    return t.to(dtype).to(torch.float64).numpy()


@pytest.mark.parametrize("fmt,dtype,frac,e_lo,e_hi,vmax", [
    (orc.P_E4M3, torch.float8_e4m3fn, 3, -12, 9, 448.0),        # subnormals below 2^-6, saturation at 448
    (orc.P_E5M2, torch.float8_e5m2, 2, -19, 16, 57344.0),       # subnormals below 2^-14, saturation at 57344
    (orc.P_BF16, torch.bfloat16, 7, -20, 20, 3.3895313892515355e38),
])
def test_p_round_matches_library_casts(fmt, dtype, frac, e_lo, e_hi, vmax):
    v = _sweep(frac, e_lo, e_hi)
    # values the fp32 step of the library route cannot tell apart from a tie are left out: the neighbours
    # at 2^-30 relative distance survive the cast to fp32 only as the tie itself
    v = np.unique(v.astype(np.float32).astype(np.float64))
    got = np.array([orc.p_round(x, fmt, 0) for x in v])
    want = _torch_cast(v, dtype, vmax)
    assert np.array_equal(got, want)
    assert orc.p_round(vmax * 4, fmt, 0) == vmax and orc.p_round(0.0, fmt, 0) == 0.0
    # the offset is an exact power-of-two scale around the rounding
    for off in (8, 15):
        w = v[(v * 2.0 ** off <= vmax)]
        got = np.array([orc.p_round(x, fmt, off) for x in w[::7]])
        assert np.array_equal(got, _torch_cast(w[::7] * 2.0 ** off, dtype, vmax) / 2.0 ** off)


def test_p_round_none_is_the_identity():
    assert orc.p_round(0.3, orc.P_NONE, 5) == 0.3


# ---- the tie-widening bound --------------------------------------------------------------------

TIE_EPS = 2.0 ** -16
# score grid on which half of the points are rounding boundaries of the mode's map
STEP = {orc.W_POT: 0.5, orc.W_H15: 0.25, orc.W_H15K2: 0.125, orc.W_H15K3: 0.0625}


def _quantity(x32, mode, kmax):
    """The number the map rounds, as the oracle's bookkeeping defines it."""
    x = x32.astype(np.float64)
    if mode == orc.W_POT:
        return -x
    k = {orc.W_H15: 1, orc.W_H15K2: 2, orc.W_H15K3: 3}[mode]
    return np.maximum(x, -126.0) * 2.0 ** k


def _flagged(x32, mode, kmax):
    u = _quantity(x32, mode, kmax)
    dist = np.abs(u - (np.floor(u) + 0.5))
    f = dist < TIE_EPS * np.maximum(1.0, np.abs(u))
    if mode == orc.W_POT:
        f &= ~(u > kmax + 1.0)
    return f


def _other_side(x32, mode, kmax, wmap):
    """Weight of each score after moving it just across its nearest rounding boundary."""
    u = _quantity(x32, mode, kmax)
    b = np.floor(u) + 0.5
    step = np.maximum(np.abs(b) * 2.0 ** -20, 2.0 ** -20)
    scale = -1.0 if mode == orc.W_POT else 2.0 ** -{orc.W_H15: 1, orc.W_H15K2: 2, orc.W_H15K3: 3}.get(mode, 0)
    below = wmap(((b - step) * scale).astype(np.float32))
    above = wmap(((b + step) * scale).astype(np.float32))
    here = wmap(x32)
    return np.where(below != here, below, above)


def _lattice_case(seed, S, tile, D=8, step=0.25):
    """Scores that are multiples of `step` octaves (c = 1): many sit exactly on a rounding boundary."""
    rng = np.random.default_rng(seed)
    q = np.zeros((1, 1, 1, D), np.float32); q[..., 0] = 1.0
    a = -rng.integers(0, int(12 / step), size=S).astype(np.float32) * np.float32(step)
    a += np.repeat(rng.integers(0, 3, size=(S + tile - 1) // tile), tile)[:S].astype(np.float32) * 0.75   # moving tile maxima
    k = np.zeros((1, S, 1, D), np.float32); k[0, :, 0, 0] = a
    v = (rng.standard_normal((1, S, 1, D)) * 2).astype(np.float32)
    v = torch.from_numpy(v).to(torch.bfloat16).float().numpy()
    return q, k, v


@pytest.mark.parametrize("mode,drop", [(orc.W_H15, False), (orc.W_POT, False), (orc.W_POT, True),
                                       (orc.W_H15K2, False), (orc.W_H15K3, False)])
def test_flipping_flagged_scores_stays_within_the_widening_bound(mode, drop):
    scale = float(np.float32(math.log(2.0)))      # c = 1
    kmax = 6 if mode == orc.W_POT else 20          # a short tail so that the drop boundary is exercised
    rng = np.random.default_rng(17)
    total_flagged = 0
    for case in range(120):
        S, tile = int(rng.integers(3, 70)), int(rng.choice([4, 16, 128]))
        q, k, v = _lattice_case(1000 + case, S, tile, step=STEP[mode])
        ref = orc.attn(_bf16_bits(q), _bf16_bits(k), _bf16_bits(v), in_dtype=orc.IN_BF16, causal=False,
                       softmax_scale=scale, mode=mode, tile_n=tile, kmax=kmax, drop_tail=drop, tie_eps=TIE_EPS)
        counted = []

        def count(x32, w, wmap):
            counted.append(int(_flagged(x32, mode, kmax).sum()))
            return w

        base_o, base_l = _numpy_online(q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), False, scale,
                                       mode, tile, kmax=kmax, drop_tail=drop, reweigh=count)
        assert np.allclose(base_o, ref["O"], rtol=1e-11, atol=1e-12)
        assert sum(counted) == int(ref["nflag"][0, 0, 0])          # the same elements are flagged
        total_flagged += sum(counted)
        for trial in range(4):
            sub = np.random.default_rng(case * 10 + trial)

            def flip(x32, w, wmap, sub=sub, trial=trial):
                f = _flagged(x32, mode, kmax)
                if trial > 0:
                    f &= sub.random(f.shape) < 0.5                 # trial 0 flips all of them
                return np.where(f, _other_side(x32, mode, kmax, wmap), w)

            o, l = _numpy_online(q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), False, scale,
                                 mode, tile, kmax=kmax, drop_tail=drop, reweigh=flip)
            d_o = np.abs(o - base_o).max()
            d_l = abs(l[0, 0, 0] - base_l[0, 0, 0])
            assert d_o <= ref["widen_o"][0, 0, 0] * (1 + 1e-9) + 1e-13, (case, trial, d_o, ref["widen_o"][0, 0, 0])
            assert d_l <= ref["widen_lse"][0, 0, 0] * (1 + 1e-9) + 1e-13, (case, trial, d_l, ref["widen_lse"][0, 0, 0])
    assert total_flagged > 300       # the cases really do sit on boundaries
