"""GPU parity of the fused attention forward against the CPU oracle, through the C interface."""
import numpy as np
import pytest
import torch

from oracle import cpu_oracle as orc
from paper_2609_33586_b200 import binding
from paper_2609_33586_b200.inputs import WORKLOADS, Workload, make_inputs

from parity_util import compare

pytestmark = pytest.mark.gpu

MODES = [orc.W_EXACT, orc.W_POT, orc.W_H15]
FAMILY = [orc.W_H15K2, orc.W_H15K3]
EXACT_POLY = binding.W_EXACT_POLY


@pytest.fixture(autouse=True)
def _device_status_is_clean():
    binding.device_status_reset()
    yield
    assert binding.device_status() == 0


@pytest.mark.parametrize("mode", MODES)
def test_config0_tiny_causal_every_row(mode):
    st = compare(WORKLOADS[0], mode)
    assert st["ok"], st


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("wl", [
    Workload("d128_ragged", 2, 4, 2, 300, 300, 128, True, "bf16", 31),       # several tiles + ragged tail
    Workload("d128_noncausal", 1, 2, 1, 257, 391, 128, False, "bf16", 32),   # Sq != Sk, not multiples of 128
    Workload("d64_cross", 1, 4, 4, 130, 520, 64, True, "bf16", 33),          # bottom-right aligned mask
    Workload("more_q_than_k", 1, 2, 2, 400, 144, 64, True, "bf16", 34),      # rows with no visible key
    Workload("one_row", 1, 1, 1, 1, 1, 128, True, "bf16", 35),               # degenerate: single query and key
    Workload("fp8_ragged", 2, 4, 2, 300, 428, 128, True, "fp8_e4m3", 36),
    Workload("fp8_noncausal", 1, 2, 2, 256, 384, 128, False, "fp8_e4m3", 37),
], ids=lambda w: w.name)
def test_small_shapes(wl, mode):
    st = compare(wl, mode)
    assert st["ok"], st


@pytest.mark.parametrize("mode", FAMILY)
@pytest.mark.parametrize("wl", [
    Workload("fam_bf16", 2, 4, 2, 300, 428, 128, True, "bf16", 51),
    Workload("fam_d64", 1, 2, 2, 257, 391, 64, False, "bf16", 52),
    Workload("fam_fp8", 2, 4, 2, 300, 428, 128, True, "fp8_e4m3", 53),
], ids=lambda w: w.name)
def test_h15_family_members_small_shapes(wl, mode):
    st = compare(wl, mode)
    assert st["ok"], st


@pytest.mark.parametrize("wl", [
    Workload("poly_bf16", 2, 4, 2, 300, 428, 128, True, "bf16", 54),
    Workload("poly_d64", 1, 2, 2, 257, 391, 64, False, "bf16", 55),
    Workload("poly_fp8", 2, 4, 2, 300, 428, 128, True, "fp8_e4m3", 56),
    WORKLOADS[0],
], ids=lambda w: w.name)
def test_partly_emulated_exact_mode_meets_the_exact_tolerances(wl):
    st = compare(wl, EXACT_POLY)
    assert st["ok"], st


@pytest.mark.parametrize("eighths", [1, 2, 3, 4])
@pytest.mark.parametrize("wl", [
    Workload("share_bf16", 2, 4, 2, 300, 428, 128, True, "bf16", 57),
    Workload("share_fp8", 1, 2, 2, 384, 384, 128, True, "fp8_e4m3", 58),
], ids=lambda w: w.name)
def test_emulation_share_of_the_exact_control(wl, eighths):
    # 12.5 to 50 % of the exponentials on the polynomial route: the exact tolerances hold for every share
    inp = make_inputs(wl)
    q, k, v = inp.q.cuda(), inp.k.cuda(), inp.v.cuda()
    o, lse = binding.attn_fwd(q, k, v, causal=wl.causal, softmax_scale=wl.softmax_scale, weight_mode=EXACT_POLY,
                              q_descale=inp.q_descale, k_descale=inp.k_descale, v_descale=inp.v_descale, poly_eighths=eighths)
    ref_o, ref_lse = binding.attn_fwd(q, k, v, causal=wl.causal, softmax_scale=wl.softmax_scale, weight_mode=orc.W_EXACT,
                                      q_descale=inp.q_descale, k_descale=inp.k_descale, v_descale=inp.v_descale)
    torch.cuda.synchronize()
    from parity_util import run_oracle, TOL
    ref = run_oracle(wl, inp, orc.W_EXACT)
    got = o.float().cpu().numpy().transpose(0, 2, 1, 3)
    tol = TOL[wl.in_dtype]["o_max"] * (2.0 if wl.in_dtype == "fp8_e4m3" else 1.0)   # causal rows with few keys: see parity_util
    assert np.abs(got - ref["O"]).max() <= tol
    assert np.abs(lse.cpu().numpy() - ref["LSE"]).max() <= 1e-3
    # and close to the plain exact mode of the same kernel
    assert (o.float() - ref_o.float()).abs().max().item() <= tol
    assert (lse - ref_lse).abs().max().item() <= 5e-4


def test_emulation_share_limits():
    q = torch.zeros(1, 128, 2, 64, dtype=torch.bfloat16, device="cuda")
    args = (q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None, 1, 2, 2, 128, 128)
    tail = (1, 0.1, EXACT_POLY, binding.IN_BF16, 1.0, 1.0, 1.0, None)
    assert binding.attn_fwd_raw(*args, 64, *tail, poly_eighths=3) == -8       # other shares: D = 128 only
    assert binding.attn_fwd_raw(*args, 64, *tail, poly_eighths=2) == 0
    assert binding.attn_fwd_raw(*args, 64, *tail, poly_eighths=5) == -9
    assert binding.attn_fwd_raw(*args, 64, *tail, poly_eighths=0) == -9
    torch.cuda.synchronize()


def test_partly_emulated_exact_mode_full_size_8k_fp8():
    wl = WORKLOADS[2]
    st = compare(wl, EXACT_POLY, rows=_sample_rows(wl.Sq, 127))
    assert st["ok"], st


@pytest.mark.parametrize("mode", FAMILY)
def test_h15_family_members_full_size_8k_fp8(mode):
    wl = WORKLOADS[2]
    st = compare(wl, mode, rows=_sample_rows(wl.Sq, 127))
    assert st["ok"], st


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        dtype = "fp8_e4m3" if rng.random() < 0.4 else "bf16"
        D = 128 if dtype == "fp8_e4m3" or rng.random() < 0.6 else 64
        hkv = int(rng.integers(1, 4))
        g = int(rng.choice([1, 2, 4]))
        B = int(rng.integers(1, 4))
        Sq = int(rng.integers(1, 700))
        Sk = int(rng.integers(1, 900))
        causal = bool(rng.random() < 0.6)
        out.append(Workload(f"fuzz{i}", B, hkv * g, hkv, Sq, Sk, D, causal, dtype, 100 + i, peaked_keys=bool(rng.random() < 0.3)))
    return out


@pytest.mark.parametrize("wl", _random_shapes(24, 7), ids=lambda w: f"{w.name}-{w.in_dtype}-B{w.B}H{w.Hq}/{w.Hkv}-{w.Sq}x{w.Sk}-D{w.D}-{'c' if w.causal else 'n'}")
def test_random_shapes_all_modes(wl):
    # ragged lengths, Sq != Sk in both directions, grouped heads, more work items than CTAs or fewer
    for mode in MODES + FAMILY + [EXACT_POLY]:
        st = compare(wl, mode, model_p_storage=True)
        assert st["ok"], (mode, st)


def test_many_work_items_per_cta():
    # 4 x 40 heads x 3 tile pairs = 480 items on 148 persistent CTAs: several rounds of the snake per CTA
    wl = Workload("many", 4, 40, 8, 700, 700, 64, True, "bf16", 61)
    st = compare(wl, orc.W_H15, rows=_sample_rows(wl.Sq, 7))
    assert st["ok"], st


@pytest.mark.parametrize("mode", [orc.W_EXACT, orc.W_H15])
def test_config1_gqa_peaked_rows(mode):
    wl = WORKLOADS[1]
    st = compare(wl, mode, rows=_sample_rows(wl.Sq, 13))
    assert st["ok"], st


def _sample_rows(S, stride):
    """Every stride-th row (strides are odd, so the samples walk through every lane and warp of the
    softmax warpgroups, in work items of every round of the persistent loop), plus all rows of the
    first and the last query tile."""
    return np.unique(np.concatenate([np.arange(0, S, stride), np.arange(128), np.arange(S - 128, S)]))


@pytest.mark.parametrize("mode", [orc.W_EXACT, orc.W_H15])
@pytest.mark.parametrize("idx", [2, 3])
def test_config2_and_3_full_size_8k_fp8_on_sampled_rows(idx, mode):
    # the workloads and launch configuration bench.py times; the oracle computes sampled rows one by one
    wl = WORKLOADS[idx]
    st = compare(wl, mode, rows=_sample_rows(wl.Sq, 61))
    assert st["ok"], st


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", ["bf16", "fp8_e4m3"])
def test_config4_full_size_16k_gqa_on_sampled_rows(dtype, mode):
    wl = WORKLOADS[4].with_(in_dtype=dtype)
    st = compare(wl, mode, rows=_sample_rows(wl.Sq, 251))
    assert st["ok"], st


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", ["bf16", "fp8_e4m3"])
def test_huge_score_range_reaches_the_clamp(mode, dtype):
    # q and k scaled by 8 (exact in both storage types): offsets from the running maximum spread over
    # hundreds of octaves, far below the h15 clamp at -126 and the pot floor at -20.
    wl = Workload("wide", 1, 2, 1, 384, 384, 128, True, dtype, 43)
    inp = make_inputs(wl)
    if dtype == "bf16":
        inp.q = (inp.q.float() * 8).to(torch.bfloat16)
        inp.k = (inp.k.float() * 8).to(torch.bfloat16)
    else:
        inp.q_descale *= 8.0
        inp.k_descale *= 8.0
    st = compare(wl, mode, inp, allow_output_rounding=True)   # rows collapse onto single values of magnitude up to 4
    assert st["ok"], st


FP16_SHAPES = [
    Workload("fp16_small", 2, 4, 2, 320, 448, 128, True, "fp16", 51),
    Workload("fp16_d64", 1, 2, 2, 384, 384, 64, False, "fp16", 52),
    Workload("fp16_peaked", 1, 4, 4, 512, 512, 128, True, "fp16", 53, peaked_keys=True),
]


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("wl", FP16_SHAPES, ids=lambda w: w.name)
def test_fp16_inputs_small_shapes(wl, mode):
    # IEEE half inputs (the FP16 rows of the timing tables in App. B); same tolerances as bf16
    st = compare(wl, mode)
    assert st["ok"], st


FP8_D64_SHAPES = [
    Workload("fp8_d64_small", 2, 4, 2, 320, 448, 64, True, "fp8_e4m3", 56),
    Workload("fp8_d64_noncausal", 1, 2, 2, 384, 384, 64, False, "fp8_e4m3", 57),
    Workload("fp8_d64_ragged", 1, 3, 1, 200, 333, 64, True, "fp8_e4m3", 58, peaked_keys=True),
]


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("wl", FP8_D64_SHAPES, ids=lambda w: w.name)
def test_fp8_head_dim_64_small_shapes(wl, mode):
    # 64-byte rows: the shared-memory tiles use the 64-byte swizzle
    st = compare(wl, mode, model_p_storage=True)
    assert st["ok"], st


@pytest.mark.parametrize("mode", [orc.W_EXACT, orc.W_H15])
def test_fp8_head_dim_64_causal_4k_on_sampled_rows(mode):
    wl = Workload("causal_4k_fp8_d64", 1, 16, 16, 4096, 4096, 64, True, "fp8_e4m3", 59)
    rows = np.unique(np.concatenate([np.arange(0, 4096, 251), [127, 128, 255, 256, 4095]])).astype(np.int32)
    st = compare(wl, mode, rows=rows)
    assert st["ok"], st


def test_fp16_inputs_reject_what_is_not_built():
    q = torch.zeros(1, 128, 2, 128, dtype=torch.float16, device="cuda")
    args = (q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None, 1, 2, 2, 128, 128, 128, 1, 0.1)
    assert binding.attn_fwd_raw(*args, binding.W_H15K2, binding.IN_FP16, 1.0, 1.0, 1.0, None) == -8
    assert binding.attn_fwd_raw(*args, binding.W_EXACT_POLY, binding.IN_FP16, 1.0, 1.0, 1.0, None) == -8
    assert binding.attn_fwd_raw(*args, binding.W_H15, binding.IN_FP16, 1.0, 1.0, 1.0, None, rescale_tau=4.0) == -8
    assert binding.get_schedule(128, binding.IN_FP16, binding.W_H15, True)["p_format"] == binding.P_FP16


@pytest.mark.parametrize("mode", [orc.W_EXACT, orc.W_H15])
def test_fp16_inputs_full_size_8k_on_sampled_rows(mode):
    wl = Workload("causal_8k_fp16", 1, 16, 16, 8192, 8192, 128, True, "fp16", 54)
    rows = np.unique(np.concatenate([np.arange(0, 8192, 509), [127, 128, 255, 256, 8191]])).astype(np.int32)
    st = compare(wl, mode, rows=rows)
    assert st["ok"], st


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("scale_up", [1.0, 2.0])
def test_h15_fp8_clamp_tests_agree(causal, scale_up):
    # The fp8 h15 path skips its row-minimum pass when 448 * sum|q_i| already keeps every offset above
    # the clamp.  scale_up = 1: the bound holds (Gaussian inputs); 2: scores four times larger, the bound
    # fails and the row minimum decides (no clamp needed yet).  Both must match the oracle; items of one
    # and of several key tiles are present (the bound is used only from two key tiles on).
    wl = Workload("floor", 1, 2, 2, 640, 640, 128, causal, "fp8_e4m3", 46)
    inp = make_inputs(wl)
    inp.q_descale *= scale_up
    inp.k_descale *= scale_up
    st = compare(wl, orc.W_H15, inp, allow_output_rounding=scale_up > 1.0)
    assert st["ok"], st


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("tau", [8.0, 2.0])
def test_deferred_rescale_matches_the_oracle_with_the_same_threshold(mode, tau):
    # the anchor lags the running maximum by up to tau octaves: x can be positive, weights exceed 1
    # (in exact mode the largest weight of a row is then 2^x with x > 0 instead of exactly 1, so its bf16
    # rounding, 2^-9 relative, shows in peaked rows: allow it on top of the bf16 rounding of O itself)
    wl = Workload("tau", 2, 4, 2, 600, 600, 128, True, "bf16", 44, peaked_keys=True)
    st = compare(wl, mode, tau=tau, allow_output_rounding=True)
    assert st["ok"], st
    wl64 = Workload("tau64", 1, 2, 2, 384, 512, 64, False, "bf16", 45)
    st = compare(wl64, mode, tau=tau, allow_output_rounding=True)
    assert st["ok"], st


def test_deferred_rescale_is_rejected_for_fp8_and_bad_values():
    q = torch.zeros(1, 128, 2, 128, dtype=torch.bfloat16, device="cuda")
    args = (q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None, 1, 2, 2, 128, 128, 128, 1, 0.1, 2)
    assert binding.attn_fwd_raw(*args, 1, 1.0, 1.0, 1.0, None, rescale_tau=8.0) == -8     # fp8
    assert binding.attn_fwd_raw(*args, 0, 1.0, 1.0, 1.0, None, rescale_tau=-1.0) == -9
    assert binding.attn_fwd_raw(*args, 0, 1.0, 1.0, 1.0, None, rescale_tau=float("nan")) == -9


@pytest.mark.parametrize("drop", [False, True])
@pytest.mark.parametrize("kmax", [8, 12, 20])
@pytest.mark.parametrize("wl", [
    Workload("pot_bf16", 2, 4, 2, 300, 428, 128, True, "bf16", 71, peaked_keys=True),
    Workload("pot_d64", 1, 2, 2, 257, 391, 64, False, "bf16", 72),
    Workload("pot_fp8", 2, 4, 2, 300, 428, 128, True, "fp8_e4m3", 73),
    Workload("pot_fp16", 1, 2, 1, 384, 384, 128, True, "fp16", 74),
], ids=lambda w: w.name)
def test_pot_tail_index_and_drop_variant(wl, kmax, drop):
    # Rowmax-PoT with the tail index K_max chosen by the caller, tail clamped or dropped (App. A, after Eq. rowmax-pot)
    inp = make_inputs(wl)
    if kmax == 8:      # spread the scores so that the short tail really cuts (offsets beyond 8 octaves are common)
        if wl.in_dtype == "fp8_e4m3":
            inp.q_descale *= 3.0
        else:
            inp.q = (inp.q.float() * 3).to(inp.q.dtype)
    st = compare(wl, orc.W_POT, inp, pot_tail=(kmax, drop), allow_output_rounding=kmax == 8)
    assert st["ok"], st


def test_pot_tail_default_is_kmax_20_clamped_and_bad_values_are_rejected():
    wl = Workload("pot_same", 1, 2, 2, 256, 256, 128, True, "bf16", 75)
    inp = make_inputs(wl)
    q, k, v = inp.q.cuda(), inp.k.cuda(), inp.v.cuda()
    a = binding.attn_fwd(q, k, v, causal=True, softmax_scale=wl.softmax_scale, weight_mode=orc.W_POT)
    b = binding.attn_fwd(q, k, v, causal=True, softmax_scale=wl.softmax_scale, weight_mode=orc.W_POT, pot_tail=(20, False))
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    args = (q.data_ptr(), k.data_ptr(), v.data_ptr(), a[0].data_ptr(), None, 1, 2, 2, 256, 256, 128, 1, 0.1, orc.W_POT)
    assert binding.attn_fwd_raw(*args, binding.IN_BF16, 1.0, 1.0, 1.0, None, pot_tail=(0, False)) == -9
    assert binding.attn_fwd_raw(*args, binding.IN_BF16, 1.0, 1.0, 1.0, None, pot_tail=(126, False)) == -9
    assert binding.attn_fwd_raw(*args, binding.IN_FP8_E4M3, 1.0, 1.0, 1.0, None, pot_tail=(30, True)) == -9
    assert binding.attn_fwd_raw(*args, binding.IN_FP16, 1.0, 1.0, 1.0, None, pot_tail=(24, False)) == -9


def test_fully_masked_rows_give_zero_and_minus_infinity():
    wl = Workload("masked", 1, 2, 2, 300, 100, 64, True, "bf16", 41)
    inp = make_inputs(wl)
    o, lse = binding.attn_fwd(inp.q.cuda(), inp.k.cuda(), inp.v.cuda(), causal=True,
                              softmax_scale=wl.softmax_scale, weight_mode=orc.W_H15)
    torch.cuda.synchronize()
    assert torch.all(o[:, :200] == 0) and torch.all(torch.isneginf(lse[:, :, :200]))
    assert torch.all(torch.isfinite(lse[:, :, 200:]))


def test_run_twice_is_bitwise_deterministic():
    wl = WORKLOADS[0].with_(Sq=512, Sk=512)
    inp = make_inputs(wl)
    q, k, v = inp.q.cuda(), inp.k.cuda(), inp.v.cuda()
    a = binding.attn_fwd(q, k, v, causal=True, softmax_scale=wl.softmax_scale, weight_mode=orc.W_H15)
    b = binding.attn_fwd(q, k, v, causal=True, softmax_scale=wl.softmax_scale, weight_mode=orc.W_H15)
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_h15_one_hot_values_expose_lattice_probabilities():
    # One-hot value rows read the kernel's normalised probabilities back (App. B "Correctness gates").
    S, D = 128, 128
    wl = Workload("onehot", 1, 1, 1, S, S, D, True, "bf16", 42)
    inp = make_inputs(wl)
    inp.v = torch.eye(S, D).reshape(1, S, 1, D).to(torch.bfloat16)
    o, _ = binding.attn_fwd(inp.q.cuda(), inp.k.cuda(), inp.v.cuda(), causal=True,
                            softmax_scale=wl.softmax_scale, weight_mode=orc.W_H15)
    p = o[0, :, 0].float().cpu().numpy()
    assert np.all(np.triu(p, 1) == 0)                       # masked keys: probability zero
    assert np.allclose(p.sum(axis=1), 1.0, atol=2e-2)       # bf16 storage of O
    ex, _ = binding.attn_fwd(inp.q.cuda(), inp.k.cuda(), inp.v.cuda(), causal=True,
                             softmax_scale=wl.softmax_scale, weight_mode=orc.W_EXACT)
    pe = ex[0, :, 0].float().cpu().numpy()
    big = np.tril(np.ones((S, S), bool)) & (pe > 1e-2)
    ratio = np.log2(p[big] / pe[big])
    assert np.all(np.abs(ratio) <= np.log2(1.5) + 0.03)     # +-0.585 octave, plus bf16 storage rounding


def test_argument_errors_are_reported_without_launching():
    before = binding.launch_count()
    q = torch.zeros(1, 128, 2, 128, dtype=torch.bfloat16, device="cuda")
    rc = binding.attn_fwd_raw(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None, 1, 2, 2, 128, 128,
                              96, 1, 0.1, 0, 0, 1.0, 1.0, 1.0, None)
    assert rc == -2                                       # D = 96
    rc = binding.attn_fwd_raw(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None, 1, 3, 2, 128, 128,
                              128, 1, 0.1, 0, 0, 1.0, 1.0, 1.0, None)
    assert rc == -2                                       # Hq % Hkv
    rc = binding.attn_fwd_raw(None, q.data_ptr(), q.data_ptr(), q.data_ptr(), None, 1, 2, 2, 128, 128, 128, 1, 0.1,
                              0, 0, 1.0, 1.0, 1.0, None)
    assert rc == -1
    rc = binding.attn_fwd_raw(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None, 1, 2, 2, 128, 128,
                              128, 1, 0.1, 9, 0, 1.0, 1.0, 1.0, None)
    assert rc == -3
    rc = binding.attn_fwd_raw(q.data_ptr() + 2, q.data_ptr(), q.data_ptr(), q.data_ptr(), None, 1, 2, 2, 64, 64,
                              128, 1, 0.1, 0, 0, 1.0, 1.0, 1.0, None)
    assert rc == -4
    rc = binding.attn_fwd_raw(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None, 1, 2, 2, 128, 128,
                              128, 1, -1.0, 0, 0, 1.0, 1.0, 1.0, None)
    assert rc == -9
    assert binding.launch_count() == before
