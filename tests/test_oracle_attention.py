"""Pins for the CPU oracle's attention functions (no GPU).

Brute force and library softmax on tiny inputs, closed forms (Q = 0, a two-key hand example),
equivalences that the mathematics fixes (one tile covering the row, integer-octave maximum
increments, GQA against expanded heads, causal against truncated keys) and the bounds the paper
states for Rowmax-H15 against exact softmax.
"""
import math

import numpy as np
import pytest
import torch

from oracle import cpu_oracle as orc
from paper_2609_33586_b200 import inputs
from paper_2609_33586_b200.inputs import Workload, make_inputs, storage_bits

LOG2_1P5 = math.log2(1.5)
LOG2E = 1.4426950408889634


def _bf16_bits(a):
    return storage_bits(torch.as_tensor(np.asarray(a, np.float32)).to(torch.bfloat16))


def _values(t):
    return t.to(torch.float64).numpy()


def _run(wl, mode, tile_n, inp=None, **kw):
    inp = inp or make_inputs(wl)
    dt = orc.IN_BF16 if wl.in_dtype == "bf16" else orc.IN_FP8_E4M3
    return orc.attn(storage_bits(inp.q), storage_bits(inp.k), storage_bits(inp.v), in_dtype=dt,
                    causal=wl.causal, softmax_scale=wl.softmax_scale, mode=mode, tile_n=tile_n,
                    q_descale=inp.q_descale, k_descale=inp.k_descale, v_descale=inp.v_descale, **kw)


TINY = Workload("t", 1, 2, 2, 40, 40, 16, True, "bf16", 11)
TINY_X = Workload("tx", 2, 4, 2, 24, 56, 16, True, "bf16", 12)   # Sq != Sk, GQA 2:1
SMALL = Workload("s", 1, 2, 1, 200, 200, 32, True, "bf16", 13)


# ---- exact mode against brute force and a library ----------------------------------------------

def _brute_force_softmax_attention(q, k, v, causal, scale):
    """Pure-Python loops over the definition: p_j = exp(s_j - max) / sum, masked entries zero."""
    B, Sq, Hq, D = q.shape
    Sk, Hkv = k.shape[1], k.shape[2]
    O = np.zeros((B, Hq, Sq, D))
    L = np.full((B, Hq, Sq), -np.inf)
    for b in range(B):
        for h in range(Hq):
            hk = h // (Hq // Hkv)
            for i in range(Sq):
                vis = [j for j in range(Sk) if (not causal) or j <= i + Sk - Sq]
                if not vis:
                    continue
                s = [scale * sum(q[b, i, h, d] * k[b, j, hk, d] for d in range(D)) for j in vis]
                m = max(s)
                w = [math.exp(x - m) for x in s]
                tot = sum(w)
                for d in range(D):
                    O[b, h, i, d] = sum(wj * v[b, j, hk, d] for wj, j in zip(w, vis)) / tot
                L[b, h, i] = m + math.log(tot)
    return O, L


@pytest.mark.parametrize("wl", [Workload("bf", 1, 2, 1, 9, 13, 8, True, "bf16", 5),
                                Workload("bf", 1, 2, 2, 10, 10, 8, False, "bf16", 6),
                                Workload("bf", 1, 2, 2, 12, 7, 8, True, "bf16", 7)])
def test_exact_matches_brute_force(wl):
    inp = make_inputs(wl)
    O, L = _brute_force_softmax_attention(_values(inp.q), _values(inp.k), _values(inp.v),
                                          wl.causal, wl.softmax_scale)
    got = _run(wl, orc.W_EXACT, 0, inp)
    assert np.allclose(got["O"], O, rtol=1e-12, atol=1e-13)
    assert np.array_equal(np.isneginf(got["LSE"]), np.isneginf(L))
    fin = np.isfinite(L)
    assert np.allclose(got["LSE"][fin], L[fin], rtol=1e-12, atol=1e-13)
    # rows that see no key (Sq > Sk, causal): O = 0, LSE = -inf
    if wl.causal and wl.Sq > wl.Sk:
        assert np.all(got["O"][:, :, : wl.Sq - wl.Sk] == 0) and np.all(np.isneginf(L[:, :, : wl.Sq - wl.Sk]))


def test_exact_matches_torch_sdpa_fp64_and_fp8_descales():
    for wl in (TINY, TINY_X.with_(causal=False), Workload("f8", 1, 4, 2, 33, 33, 16, True, "fp8_e4m3", 3)):
        inp = make_inputs(wl)
        q = inp.q.to(torch.float64) * inp.q_descale
        k = inp.k.to(torch.float64) * inp.k_descale
        v = inp.v.to(torch.float64) * inp.v_descale
        g = wl.Hq // wl.Hkv
        k = k.repeat_interleave(g, dim=2)
        v = v.repeat_interleave(g, dim=2)
        ref = torch.nn.functional.scaled_dot_product_attention(
            q.transpose(1, 2), k.transpose(1, 2), v.transpose(1, 2), is_causal=wl.causal,
            scale=wl.softmax_scale)
        got = _run(wl, orc.W_EXACT, 0, inp)
        assert np.allclose(got["O"], ref.numpy(), rtol=1e-10, atol=1e-12)


def test_online_exact_agrees_with_definition():
    ref = _run(SMALL, orc.W_EXACT, 0)
    for tile, order in ((16, 1), (64, -1), (128, 1)):
        on = _run(SMALL, orc.W_EXACT, tile, kv_order=order)
        # x is rounded to fp32 in the online loop, hence ~1e-7 relative
        assert np.allclose(on["O"], ref["O"], rtol=0, atol=5e-6)
        assert np.allclose(on["LSE"], ref["LSE"], rtol=0, atol=5e-6)


# ---- closed forms that hold in every mode ------------------------------------------------------

@pytest.mark.parametrize("mode", [orc.W_EXACT, orc.W_POT, orc.W_H15])
def test_zero_queries_give_the_mean_of_visible_values(mode):
    wl = TINY_X
    inp = make_inputs(wl)
    inp.q = torch.zeros_like(inp.q)
    got = _run(wl, mode, 16, inp)
    v = _values(inp.v)
    for b in range(wl.B):
        for h in range(wl.Hq):
            for i in range(wl.Sq):
                nvis = i + wl.Sk - wl.Sq + 1
                want = v[b, :nvis, h // 2].mean(axis=0)
                assert np.allclose(got["O"][b, h, i], want, rtol=1e-12, atol=1e-14)
                assert abs(got["LSE"][b, h, i] - math.log(nvis)) < 1e-12


def test_two_key_hand_example():
    # scale = ln 2 makes c = 1; q.k0 - q.k1 = 1.5, so the second key sits 1.5 octaves below the max:
    # exact 2^-1.5, pot 2^-2 (tie goes up in d), h15 1.5 * 2^-2 (the paper's n = -3 example).
    D = 8
    q = np.zeros((1, 1, 1, D), np.float32); q[..., 0] = 1.0
    k = np.zeros((1, 2, 1, D), np.float32); k[0, 0, 0, 0] = 2.0; k[0, 1, 0, 0] = 0.5
    v = np.zeros((1, 2, 1, D), np.float32); v[0, 0, 0, :] = 1.0; v[0, 1, 0, :] = -3.0
    # ln 2 is not an fp32-exact scale times log2 e = 1; pick c exactly: scale = 1/log2(e) in fp32
    scale = float(np.float32(1.0 / LOG2E))
    c = float(np.float32(scale * LOG2E))
    assert abs(c - 1.0) < 1e-7
    for mode, w1 in ((orc.W_EXACT, 2.0 ** (-1.5 * c)), (orc.W_POT, 0.25), (orc.W_H15, 0.375)):
        got = orc.attn(_bf16_bits(q), _bf16_bits(k), _bf16_bits(v), in_dtype=orc.IN_BF16,
                       causal=False, softmax_scale=scale, mode=mode, tile_n=128)
        want_o = (1.0 + w1 * -3.0) / (1.0 + w1)
        assert np.allclose(got["O"][0, 0, 0], want_o, rtol=1e-6), (mode, got["O"][0, 0, 0, 0], want_o)
        want_lse = math.log(2.0) * (2.0 * c + math.log2(1.0 + w1))
        assert abs(got["LSE"][0, 0, 0] - want_lse) < 1e-6


# ---- a second, independent coding of the online loop -------------------------------------------

def _numpy_online(q, k, v, causal, scale, mode, tile_n, order=1, tau=0.0, kmax=20, drop_tail=False, reweigh=None):
    """NumPy restatement of the online loop (running maximum per key tile, rescale, shared weights
    for the row sum and PV), vectorised over the tile and coded separately from the C oracle.
    `reweigh(x32, w)` may replace the weights of a tile (used to move scores across a rounding boundary)."""
    B, Sq, Hq, D = q.shape
    Sk, Hkv = k.shape[1], k.shape[2]
    c = np.float32(scale * LOG2E)
    cd = float(c)
    O = np.zeros((B, Hq, Sq, D)); L = np.full((B, Hq, Sq), -np.inf)

    def wmap(x32):
        x = x32.astype(np.float64)
        if mode == orc.W_EXACT:
            return np.exp2(x)
        if mode == orc.W_POT:
            d = np.floor(-x + 0.5)
            return np.where((d > kmax) & drop_tail, 0.0, np.exp2(-np.minimum(kmax, d)))
        if mode in (orc.W_H15K2, orc.W_H15K3):
            st = 4.0 if mode == orc.W_H15K2 else 8.0
            q = np.rint(st * np.maximum(x, -126.0)) / st
            return np.exp2(np.floor(q)) * (1.0 + q - np.floor(q))
        n = np.rint(2.0 * np.maximum(x, -126.0))
        return np.where(n % 2 == 0, 1.0, 1.5) * np.exp2(np.floor(n / 2.0))

    for b in range(B):
        for h in range(Hq):
            hk = h // (Hq // Hkv)
            for i in range(Sq):
                nvis = min(Sk, i + Sk - Sq + 1) if causal else Sk
                if nvis <= 0:
                    continue
                z = k[b, :nvis, hk] @ q[b, i, h]
                tiles = [(a, min(a + tile_n, nvis)) for a in range(0, nvis, tile_n)]
                if order < 0:
                    tiles = tiles[::-1]
                m, l, acc = -np.inf, 0.0, np.zeros(D)
                for a, e in tiles:
                    mt = z[a:e].max()
                    if m == -np.inf or (mt - m) * cd > tau:
                        mn = max(m, mt)
                        alpha = 0.0 if m == -np.inf else 2.0 ** ((m - mn) * cd)
                        l *= alpha; acc *= alpha; m = mn
                    mc = float(np.float32(m * cd))
                    x32 = (z[a:e] * cd - mc).astype(np.float32)
                    w = wmap(x32)
                    if reweigh is not None:
                        w = reweigh(x32, w, wmap)
                    l += w.sum(); acc += w @ v[b, a:e, hk]
                O[b, h, i] = acc / l
                L[b, h, i] = math.log(2.0) * (m * cd + math.log2(l))
    return O, L


@pytest.mark.parametrize("mode", [orc.W_EXACT, orc.W_POT, orc.W_H15, orc.W_H15K2, orc.W_H15K3])
@pytest.mark.parametrize("tile_n,order,tau", [(16, 1, 0.0), (16, -1, 0.0), (8, 1, 3.0)])
def test_online_matches_independent_numpy_coding(mode, tile_n, order, tau):
    wl = TINY_X
    inp = make_inputs(wl)
    O, L = _numpy_online(_values(inp.q), _values(inp.k), _values(inp.v), wl.causal,
                         wl.softmax_scale, mode, tile_n, order, tau)
    got = _run(wl, mode, tile_n, inp, kv_order=order, tau=tau)
    assert np.allclose(got["O"], O, rtol=1e-11, atol=1e-12)
    assert np.allclose(got["LSE"], L, rtol=1e-11, atol=1e-12)


# ---- the deferred rescale (threshold tau > 0) against what the mathematics fixes ----------------

@pytest.mark.parametrize("tau", [2.0, 8.0])
@pytest.mark.parametrize("tile_n", [8, 16, 128])
def test_exact_mode_does_not_depend_on_the_rescale_threshold(tau, tile_n):
    # With w = 2^x the anchor cancels between numerator and denominator: any adoption rule gives the
    # softmax of the definition, in O and in LSE.
    for wl in (TINY_X, SMALL):
        inp = make_inputs(wl)
        want = _run(wl, orc.W_EXACT, 0, inp)
        got = _run(wl, orc.W_EXACT, tile_n, inp, tau=tau)
        assert np.allclose(got["O"], want["O"], rtol=0, atol=2e-7)      # x is rounded to fp32 in the loop
        assert np.allclose(got["LSE"], want["LSE"], rtol=0, atol=2e-6)


def test_lagging_anchor_hand_example():
    # One query, four keys, tiles of ONE key, c = 1, tau = 1.  Scores 0, 0.5, 1, 3 octaves.
    #   key 0: first tile, anchor m = 0, x = 0                      -> every map gives 1
    #   key 1: 0.5 above the anchor, not more than tau: m stays 0, x = +0.5
    #          h15: n = RNE(1) = 1 -> 1.5 (Eq. h15 covers positive x); pot: floor(-0.5 + 0.5) = 0 -> 1; exact: 2^0.5
    #   key 2: 1.0 above, still not MORE than tau: x = +1 -> h15 2, pot 2^-floor(-0.5) = 2, exact 2
    #   key 3: 3.0 above > tau: adopted, alpha = 2^-3, x = 0 -> 1
    D = 8
    q = np.zeros((1, 1, 1, D), np.float32); q[..., 0] = 1.0
    k = np.zeros((1, 4, 1, D), np.float32); k[0, :, 0, 0] = [0.0, 0.5, 1.0, 3.0]
    v = np.zeros((1, 4, 1, D), np.float32); v[0, :, 0, 0] = [1.0, -2.0, 4.0, 8.0]; v[0, :, 0, 1] = 1.0
    scale = float(np.float32(math.log(2.0)))       # c = fl32(ln2 * log2 e) = 1 exactly
    for mode, w1, w2 in ((orc.W_H15, 1.5, 2.0), (orc.W_POT, 1.0, 2.0), (orc.W_EXACT, 2.0 ** 0.5, 2.0)):
        got = orc.attn(_bf16_bits(q), _bf16_bits(k), _bf16_bits(v), in_dtype=orc.IN_BF16, causal=False,
                       softmax_scale=scale, mode=mode, tile_n=1, tau=1.0)
        l = (1.0 + w1 + w2) / 8.0 + 1.0
        want0 = ((1.0 * 1.0 + w1 * -2.0 + w2 * 4.0) / 8.0 + 8.0) / l
        assert abs(got["O"][0, 0, 0, 0] - want0) < 1e-12, (mode, got["O"][0, 0, 0, 0], want0)
        assert abs(got["O"][0, 0, 0, 1] - 1.0) < 1e-12
        assert abs(got["LSE"][0, 0, 0] - math.log(2.0) * (3.0 + math.log2(l))) < 1e-12
    # tau = 0 on the same input: every tile is adopted, every x is 0, the rescales carry the differences
    got = orc.attn(_bf16_bits(q), _bf16_bits(k), _bf16_bits(v), in_dtype=orc.IN_BF16, causal=False,
                   softmax_scale=scale, mode=orc.W_H15, tile_n=1, tau=0.0)
    l = ((1.0 * 2.0 ** -0.5 + 1.0) * 2.0 ** -0.5 + 1.0) * 0.25 + 1.0
    assert abs(got["LSE"][0, 0, 0] - math.log(2.0) * (3.0 + math.log2(l))) < 1e-12


# ---- equivalences fixed by the mathematics -----------------------------------------------------

def _whole_row(wl, inp, mode):
    """Whole-row operator: anchor = the row's true maximum, weights from the map, no tiles."""
    return _numpy_online(_values(inp.q), _values(inp.k), _values(inp.v), wl.causal,
                         wl.softmax_scale, mode, tile_n=10 ** 9)


@pytest.mark.parametrize("mode", [orc.W_POT, orc.W_H15])
def test_single_tile_equals_whole_row_and_tiling_changes_the_result(mode):
    wl = SMALL
    inp = make_inputs(wl)
    O, L = _whole_row(wl, inp, mode)
    one = _run(wl, mode, 256, inp)            # one tile covers every row
    assert np.allclose(one["O"], O, rtol=1e-11, atol=1e-12)
    tiled = _run(wl, mode, 32, inp)
    # the running-maximum anchor is not the whole-row anchor: results differ measurably
    assert np.abs(tiled["O"] - O).max() > 1e-3


def test_integer_octave_increments_make_online_equal_whole_row():
    # Build scores whose tile maxima rise by whole octaves: k_j = a_j * e0 with q = e0 and c = 1.
    D, S, T = 8, 64, 16
    rng = np.random.default_rng(3)
    q = np.zeros((1, 1, 1, D), np.float32); q[..., 0] = 1.0
    a = -rng.integers(1, 6, size=S).astype(np.float32) - rng.integers(0, 8, size=S) / 8.0
    for t in range(S // T):          # tile t has the exact maximum 2 t (an integer)
        a[t * T + int(rng.integers(0, T))] = 0.0
        a[t * T:(t + 1) * T] += 2.0 * t
    k = np.zeros((1, S, 1, D), np.float32); k[0, :, 0, 0] = a
    v = rng.standard_normal((1, S, 1, D)).astype(np.float32)
    scale = float(np.float32(1.0 / LOG2E))
    for mode in (orc.W_POT, orc.W_H15):
        kw = dict(in_dtype=orc.IN_BF16, causal=False, softmax_scale=scale, mode=mode)
        on = orc.attn(_bf16_bits(q), _bf16_bits(k), _bf16_bits(v), tile_n=T, **kw)
        whole = orc.attn(_bf16_bits(q), _bf16_bits(k), _bf16_bits(v), tile_n=S, **kw)
        assert np.allclose(on["O"], whole["O"], rtol=1e-6, atol=1e-7)
        assert np.allclose(on["LSE"], whole["LSE"], rtol=1e-6, atol=1e-7)


@pytest.mark.parametrize("mode", [orc.W_EXACT, orc.W_H15])
def test_gqa_equals_expanded_heads_and_causal_equals_truncation(mode):
    wl = TINY_X
    inp = make_inputs(wl)
    tile = 0 if mode == orc.W_EXACT else 16
    got = _run(wl, mode, tile, inp)
    g = wl.Hq // wl.Hkv
    exp_inp = inputs.Inputs(inp.q, inp.k.repeat_interleave(g, dim=2), inp.v.repeat_interleave(g, dim=2), 1, 1, 1)
    full = _run(wl.with_(Hkv=wl.Hq), mode, tile, exp_inp)
    assert np.array_equal(got["O"], full["O"]) and np.array_equal(got["LSE"], full["LSE"])
    # causal row i == non-causal attention over the first i + Sk - Sq + 1 keys
    for i in (0, 7, wl.Sq - 1):
        nvis = i + wl.Sk - wl.Sq + 1
        cut = inputs.Inputs(inp.q, inp.k[:, :nvis].contiguous(), inp.v[:, :nvis].contiguous(), 1, 1, 1)
        nc = _run(wl.with_(Sk=nvis, causal=False), mode, tile, cut, rows=[i])
        assert np.allclose(nc["O"][:, :, 0], got["O"][:, :, i], rtol=1e-13, atol=0)


def test_row_subset_and_thread_count_do_not_change_results():
    full = _run(SMALL, orc.W_H15, 32, nthreads=1)
    sub = _run(SMALL, orc.W_H15, 32, rows=[0, 5, 199], nthreads=3)
    assert sub["threads"] == 3 and full["threads"] == 1
    assert np.array_equal(sub["O"], full["O"][:, :, [0, 5, 199]])
    assert np.array_equal(sub["LSE"], full["LSE"][:, :, [0, 5, 199]])


# ---- the paper's bounds for H15 against exact softmax ------------------------------------------

def test_h15_probabilities_within_bounds_of_exact_via_one_hot_values():
    # One-hot value rows expose the normalised probabilities (App. B "Correctness gates").
    S, D = 64, 64
    wl = Workload("g", 1, 1, 1, S, S, D, True, "bf16", 21)
    inp = make_inputs(wl)
    inp.v = torch.eye(S, D).reshape(1, S, 1, D).to(torch.bfloat16)
    p_exact = _run(wl, orc.W_EXACT, 0, inp)
    for tile in (64, 16):
        p_h15 = _run(wl, orc.W_H15, tile, inp)
        pe, ph = p_exact["O"][0, 0], p_h15["O"][0, 0]
        assert np.allclose(ph.sum(axis=1), 1.0, atol=1e-12)          # normalised rows
        vis = np.tril(np.ones((S, S), bool))
        assert np.all(ph[~vis] == 0)                                  # masked keys: probability zero
        ratio = np.log2(ph[vis] / pe[vis])
        width = LOG2_1P5                                              # [a - b, b - a] = +-0.585
        assert ratio.min() >= -width - 1e-6 and ratio.max() <= width + 1e-6
        dl = (p_h15["LSE"] - p_exact["LSE"]) / math.log(2.0)          # log2 of the row-sum ratio
        assert dl.min() >= -0.25 - 1e-6 and dl.max() <= LOG2_1P5 - 0.25 + 1e-6
    # with a single tile the weight at the row maximum is exactly 1, so the largest probability of
    # each row is 1 / l and every other probability is a lattice multiple of it
    one = _run(wl, orc.W_H15, 64, inp)["O"][0, 0]
    rel = one / one.max(axis=1, keepdims=True)
    mant, _ = np.frexp(rel[rel > 0])
    assert np.all(np.isclose(mant, 0.5, atol=1e-12) | np.isclose(mant, 0.75, atol=1e-12))


def test_outputs_lie_in_the_convex_hull_of_visible_values():
    wl = SMALL
    inp = make_inputs(wl)
    v = _values(inp.v)[0, :, 0]
    for mode in (orc.W_POT, orc.W_H15):
        got = _run(wl, mode, 32, inp)["O"][0]
        for i in (0, 1, 50, 199):
            lo, hi = v[: i + 1].min(axis=0), v[: i + 1].max(axis=0)
            assert np.all(got[:, i] >= lo - 1e-12) and np.all(got[:, i] <= hi + 1e-12)


def test_scale_identity():
    # Doubling softmax_scale equals doubling q (exactly representable), in every mode.
    wl = TINY
    inp = make_inputs(wl)
    dbl = inputs.Inputs((inp.q.float() * 2).to(torch.bfloat16), inp.k, inp.v, 1, 1, 1)
    for mode, tile in ((orc.W_EXACT, 0), (orc.W_H15, 16), (orc.W_POT, 16)):
        a = orc.attn(storage_bits(dbl.q), storage_bits(inp.k), storage_bits(inp.v), in_dtype=orc.IN_BF16,
                     causal=True, softmax_scale=wl.softmax_scale, mode=mode, tile_n=tile)
        b = orc.attn(storage_bits(inp.q), storage_bits(inp.k), storage_bits(inp.v), in_dtype=orc.IN_BF16,
                     causal=True, softmax_scale=2 * wl.softmax_scale, mode=mode, tile_n=tile)
        assert np.allclose(a["O"], b["O"], rtol=1e-12, atol=1e-13)


# ---- diagnostics owned by this build (tie bookkeeping, P rounding) -----------------------------

def test_tie_bookkeeping_flags_elements_on_a_rounding_boundary():
    D = 8
    q = np.zeros((1, 1, 1, D), np.float32); q[..., 0] = 1.0
    k = np.zeros((1, 3, 1, D), np.float32); k[0, :, 0, 0] = [0.0, -0.75, -1.0]   # 2x = -1.5 is a tie
    v = np.ones((1, 3, 1, D), np.float32)
    scale = float(np.float32(1.0 / LOG2E))
    got = orc.attn(_bf16_bits(q), _bf16_bits(k), _bf16_bits(v), in_dtype=orc.IN_BF16, causal=False,
                   softmax_scale=scale, mode=orc.W_H15, tile_n=128, tie_eps=2.0 ** -16)
    assert got["nflag"][0, 0, 0] == 1 and got["widen_o"][0, 0, 0] > 0 and got["widen_lse"][0, 0, 0] > 0
    none = orc.attn(_bf16_bits(q), _bf16_bits(k), _bf16_bits(v), in_dtype=orc.IN_BF16, causal=False,
                    softmax_scale=scale, mode=orc.W_EXACT, tile_n=128, tie_eps=2.0 ** -16)
    assert none["nflag"].sum() == 0


def test_p_round_leaves_lattice_weights_unchanged_where_they_are_representable():
    wl = SMALL
    base = _run(wl, orc.W_H15, 32)
    assert np.array_equal(_run(wl, orc.W_H15, 32, p_round=orc.P_BF16)["O"], base["O"])
    # e5m2 with a 2^15 offset holds {1,1.5} * 2^k exactly down to k = -29
    e5 = _run(wl, orc.W_H15, 32, p_round=orc.P_E5M2, p_off=15)
    assert np.allclose(e5["O"], base["O"], rtol=0, atol=1e-7)
    # exact-mode weights do change under e4m3 rounding (3 fraction bits)
    ex = _run(wl, orc.W_EXACT, 32)
    ex8 = _run(wl, orc.W_EXACT, 32, p_round=orc.P_E4M3, p_off=8)
    assert 1e-4 < np.abs(ex8["O"] - ex["O"]).max() < 0.2


def test_bad_arguments_are_rejected():
    z = np.zeros((1, 4, 2, 8), np.uint16)
    with pytest.raises(ValueError):
        orc.attn(z, z[:, :, :1].repeat(3, axis=2), z, in_dtype=orc.IN_BF16, causal=False,
                 softmax_scale=1.0, mode=orc.W_EXACT)           # Hq % Hkv != 0 (2 % 3)
    with pytest.raises(ValueError):
        orc.attn(z, z, z, in_dtype=orc.IN_BF16, causal=False, softmax_scale=1.0, mode=orc.W_H15, tile_n=0)
    with pytest.raises(TypeError):
        orc.attn(z.astype(np.uint8), z, z, in_dtype=orc.IN_BF16, causal=False, softmax_scale=1.0, mode=0)
