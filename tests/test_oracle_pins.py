"""Pins of the CPU oracle against what the paper and the mathematics fix.

Each test checks one function of ``oracle/baoc_oracle.py`` against a closed
form, an invariant, a library routine that a special case reduces to, or
brute force, chosen so that a dropped term, a wrong sign or a transposed
operand fails at least one of them.  No GPU is needed.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import baoc_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def _gold():
    out = {}
    for line in open(GOLD):
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split()
            out[k] = float(v)
    return out


RNG = np.random.default_rng(1234)


def _run_window(gs, o=None):
    o = o or O.Opts()
    st = O.stats_init(gs[0].shape[0])
    for g in gs:
        O.stats_step(st, g, o)
    return st


# ---------------------------------------------------------------- constants

def test_defaults_match_paper_constants():
    g, o = _gold(), O.Opts()
    assert o.eps == g["eps"]
    assert o.a_lo == math.log(g["A_low_ratio"]) and o.a_hi == math.log(g["A_high_ratio"])
    assert (o.rho_lo, o.rho_hi, o.snr_lo, o.snr_hi) == (g["rho_low"], g["rho_high"], g["snr_low"], g["snr_high"])
    assert o.gamma == g["gamma"]
    assert o.w == (1.0,) * 5 and (o.beta_m, o.beta_v) == (0.9, 0.999)


# ---------------------------------------------------------------- P1 stability (Eq. 5 left)

def test_stability_identical_gradients_is_one():
    g = RNG.standard_normal(1000)
    st = _run_window([g] * 6)
    assert abs(st.rho_bar - 1.0) <= 1e-12 / np.dot(g, g) + 1e-15
    assert st.n_cos == 5


def test_stability_sign_flip_and_zero():
    g = RNG.standard_normal(513)
    st = _run_window([g, -g, g, -g])
    assert abs(st.rho_bar + 1.0) < 1e-12
    st = _run_window([np.zeros(64)] * 4)
    assert st.rho_bar == 0.0
    st = _run_window([g])                     # a window of one step has no cosine
    assert st.rho_bar == 0.0 and st.n_cos == 0


def test_stability_orthogonal_and_ema_recursion():
    e0, e1 = np.eye(4)[0], np.eye(4)[1]
    d = (e0 + e1) / math.sqrt(2.0)
    # cosines in order: <e1,e0>=0, <d,e1>=1/sqrt2, <d,d>=1
    st = _run_window([e0, e1, d, d])
    c = [0.0, 1 / math.sqrt(2.0), 1.0]
    want = c[0]
    for x in c[1:]:
        want = 0.9 * want + 0.1 * x
    assert abs(st.rho_bar - want) < 1e-12
    assert abs(st.last_cos - 1.0) < 1e-11


def test_cosine_is_scale_invariant_and_uses_both_norms():
    a, b = RNG.standard_normal(300), RNG.standard_normal(300)
    st1 = _run_window([a, b])
    st2 = _run_window([7.0 * a, 0.01 * b])
    assert abs(st1.rho_bar - st2.rho_bar) < 1e-9
    ref = float(a @ b / (np.linalg.norm(a) * np.linalg.norm(b)))
    assert abs(st1.rho_bar - ref) < 1e-9


def test_momentum_cosine_uses_previous_moment():
    a, b = RNG.standard_normal(100), RNG.standard_normal(100)
    st = _run_window([a, b])
    # m after step 1 is 0.1*a, so cos(b, m_prev) = cos(b, a)
    assert abs(st.rho_mom - st.rho_bar) < 1e-9


# ---------------------------------------------------------------- P2 moments and SNR (Eq. 3, Eq. 5 right)

@pytest.mark.parametrize("T", [1, 5, 32])
def test_constant_gradient_closed_forms(T):
    o = O.Opts()
    g = RNG.standard_normal(257)
    st = _run_window([g] * T, o)
    np.testing.assert_allclose(st.m, (1 - o.beta_m ** T) * g, rtol=1e-12)
    np.testing.assert_allclose(st.v, (1 - o.beta_v ** T) * g * g, rtol=1e-12)
    want = (1 - o.beta_m ** T) ** 2 / (1 - o.beta_v ** T)
    assert abs(O.snr(st.m, st.v, o.eps) / want - 1.0) < 1e-9


@pytest.mark.parametrize("T", [1, 5, 32])
def test_debiased_window_moments_closed_forms(T):
    """The alternative reading of the hats in Eq. 3 (Opts.debias): a constant gradient g gives m / (1 - beta_m^T) = g and
    v / (1 - beta_v^T) = g^2 exactly, so the diagnostics are those of (g, g^2): SNR = sum g^2 / (sum g^2 + eps), every
    element of the direction has modulus |g| / (|g| + eps_adam), and the quantiles are those of g^2.  With the option
    off the same window gives the raw closed forms of the test above: the two readings differ."""
    o = O.Opts(debias=True)
    g = RNG.standard_normal(257)
    st = _run_window([g] * T, o)
    m, v = O.window_moments(st, o)
    np.testing.assert_allclose(m, g, rtol=1e-12)
    np.testing.assert_allclose(v, g * g, rtol=1e-12)
    raw = O.stats_finalize(st, np.ones(257), 257, 1, o)
    s2 = float(np.sum(g * g))
    assert abs(raw["snr"] / (s2 / (s2 + o.eps)) - 1.0) < 1e-9
    assert abs(raw["q10"] / np.quantile(g * g, 0.1) - 1.0) < 1e-9 and abs(raw["q90"] / np.quantile(g * g, 0.9) - 1.0) < 1e-9
    assert abs(raw["A"] - math.log((np.quantile(g * g, 0.9) + o.eps) / (np.quantile(g * g, 0.1) + o.eps))) < 1e-9
    off = O.stats_finalize(st, np.ones(257), 257, 1, O.Opts())
    want_off = (1 - o.beta_m ** T) ** 2 / (1 - o.beta_v ** T)
    assert abs(off["snr"] / want_off - 1.0) < 1e-9
    if T > 1:
        assert abs(off["snr"] - raw["snr"]) > 1e-3
    # the correction is a positive rescaling of each moment: the anisotropy of Eq. 4 changes only through eps
    assert abs(off["A"] - raw["A"]) < 1e-6


def test_debias_uses_the_steps_observed_and_leaves_an_empty_window_alone():
    o = O.Opts(debias=True)
    st = O.stats_init(4)
    m, v = O.window_moments(st, o)
    assert np.all(m == 0.0) and np.all(v == 0.0)                 # no step, no division by 1 - beta^0 = 0
    g1, g2 = np.array([1.0, -2.0, 0.5, 4.0]), np.array([0.0, 1.0, -1.0, 2.0])
    O.stats_step(st, g1, o); O.stats_step(st, g2, o)
    m, v = O.window_moments(st, o)
    bm, bv = o.beta_m, o.beta_v
    np.testing.assert_allclose(m, ((1 - bm) * bm * g1 + (1 - bm) * g2) / (1 - bm ** 2), rtol=1e-14)
    np.testing.assert_allclose(v, ((1 - bv) * bv * g1 ** 2 + (1 - bv) * g2 ** 2) / (1 - bv ** 2), rtol=1e-14)


def test_moments_match_explicit_weighted_sums():
    o = O.Opts()
    gs = [RNG.standard_normal(50) for _ in range(7)]
    st = _run_window(gs, o)
    T = len(gs)
    m = sum((1 - o.beta_m) * o.beta_m ** (T - 1 - k) * gs[k] for k in range(T))
    v = sum((1 - o.beta_v) * o.beta_v ** (T - 1 - k) * gs[k] ** 2 for k in range(T))
    np.testing.assert_allclose(st.m, m, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(st.v, v, rtol=1e-12, atol=1e-15)


def test_snr_uses_l1_of_v_and_squared_l2_of_m():
    m = np.array([3.0, -4.0])
    v = np.array([2.0, 6.0])
    assert abs(O.snr(m, v, 0.0) - 25.0 / 8.0) < 1e-15


# ---------------------------------------------------------------- P3 anisotropy and quantiles (Eq. 4)

def test_isotropic_gradient_has_zero_anisotropy():
    o = O.Opts()
    s = RNG.choice([-1.0, 1.0], size=999) * 0.37
    st = _run_window([s, -s, s], o)
    assert abs(O.anisotropy(st.v, o.eps)) < 1e-9


def test_two_level_vector_gives_log_ratio():
    v = np.concatenate([np.full(500, 2.0), np.full(500, 32.0)])
    RNG.shuffle(v)
    assert abs(O.anisotropy(v, 0.0) - math.log(16.0)) < 1e-12
    # eps enters both numerator and denominator
    assert abs(O.anisotropy(np.array([0.0, 0.0, 1.0, 1.0]), 0.5) - math.log(1.5 / 0.5)) < 1e-12


@pytest.mark.parametrize("n", [1, 2, 3, 10, 11, 257, 1000])
@pytest.mark.parametrize("q", [0.1, 0.9, 0.5])
def test_quantile_matches_numpy_and_torch(n, q):
    x = RNG.standard_normal(n) ** 2
    assert abs(O.quantile_linear(x, q) - np.quantile(x, q)) <= 1e-12 * max(1.0, abs(np.quantile(x, q)))
    tq = torch.quantile(torch.from_numpy(x), q).item()
    assert abs(O.quantile_linear(x, q) - tq) <= 1e-12 * max(1.0, abs(tq))


def test_quantile_hand_example():
    # positions 0.1*4 = 0.4 and 0.9*4 = 3.6 over the sorted values 1 2 3 4 5
    x = np.array([5.0, 1.0, 4.0, 2.0, 3.0])
    assert abs(O.quantile_linear(x, 0.1) - 1.4) < 1e-12
    assert abs(O.quantile_linear(x, 0.9) - 4.6) < 1e-12


# ---------------------------------------------------------------- distortion (Eq. 6)

def test_distortion_zero_for_constant_preconditioner():
    theta = RNG.standard_normal(400)
    assert O.distortion(np.full(400, 0.3), theta, 1e-12) < 1e-12


def test_distortion_hand_example():
    # sqrt(v) = (1, 3) -> p = (1, 1/3), mean 2/3, p/pbar - 1 = (1/2, -1/2)
    v = np.array([1.0, 9.0])
    theta = np.array([2.0, -4.0])
    want = math.sqrt(1.0 + 4.0) / math.sqrt(20.0)
    assert abs(O.distortion(v, theta, 0.0) - want) < 1e-12


def test_distortion_is_invariant_to_scaling_theta_and_v():
    v = RNG.standard_normal(300) ** 2 + 0.1
    th = RNG.standard_normal(300)
    a = O.distortion(v, th, 0.0)
    assert abs(O.distortion(16.0 * v, 3.0 * th, 0.0) - a) < 1e-12


# ---------------------------------------------------------------- P4 structure residual (Eq. 7)

def test_rank_one_second_moment_has_zero_residual():
    x, y = RNG.random(37) + 0.1, RNG.random(53) + 0.1
    assert O.structure_residual(np.outer(x, y).reshape(-1), 37, 53, 1e-12) < 1e-12


def test_identity_like_residual_closed_form():
    # S = I_n: row and column means 1/n, mu = 1/n, so S~ = (1/n)(1/n)/(1/n) = 1/n everywhere.
    n = 6
    want = math.sqrt(n * (1 - 1 / n) ** 2 + (n * n - n) / n ** 2) / math.sqrt(n)
    assert abs(O.structure_residual(np.eye(n).reshape(-1), n, n, 0.0) - want) < 1e-12


def test_structure_residual_depends_on_shape_orientation():
    S = RNG.random((8, 12))
    S[2, 5] += 5.0
    a = O.structure_residual(S.reshape(-1), 8, 12, 0.0)
    b = O.structure_residual(S.T.copy().reshape(-1), 12, 8, 0.0)
    assert abs(a - b) < 1e-12                       # transposing the matrix AND the shape: same residual
    c = O.structure_residual(S.reshape(-1), 12, 8, 0.0)
    assert abs(a - c) > 1e-3                        # wrong shape for the same buffer: different
    assert O.structure_residual(RNG.random(10), 10, 1, 0.0) == 1.0


# ---------------------------------------------------------------- P8 quantisers and precision cosine (Eq. 8)

def test_quantize8_roundtrip_of_representable_values_is_exact():
    a = np.float32(0.7316)
    codes = RNG.integers(-127, 128, size=700)
    codes[5] = 127                                   # make the absmax of every block equal to a
    codes[300] = -127
    codes[600] = 127
    x = codes.astype(np.float64) * float(a) / 127.0
    c, am = O.quantize8(x, True)
    np.testing.assert_array_equal(c, codes.astype(np.int8))
    np.testing.assert_array_equal(am, np.full(3, a, np.float32))
    np.testing.assert_allclose(O.dequantize8(c, am, True), x, rtol=0, atol=0)
    cu = RNG.integers(0, 256, size=512)
    cu[0] = 255
    cu[256] = 255
    xu = cu.astype(np.float64) * float(a) / 255.0
    c2, a2 = O.quantize8(xu, False)
    np.testing.assert_array_equal(c2, cu.astype(np.uint8))
    np.testing.assert_allclose(O.dequantize8(c2, a2, False), xu, rtol=0, atol=0)


def test_quantize8_error_bound_and_ragged_tail():
    x = RNG.standard_normal(1000)
    c, a = O.quantize8(x, True)
    assert a.shape == (4,) and c.dtype == np.int8
    xr = O.dequantize8(c, a, True)
    bound = np.repeat(a.astype(np.float64), 256)[:1000] / 254.0
    assert np.all(np.abs(x - xr) <= bound * (1 + 1e-6))
    v = x * x
    cv, av = O.quantize8(v, False)
    vr = O.dequantize8(cv, av, False)
    boundv = np.repeat(av.astype(np.float64), 256)[:1000] / 510.0
    assert np.all(np.abs(v - vr) <= boundv * (1 + 1e-6))
    # absmax is per block of 256 consecutive elements, the last one short
    assert a[3] == np.float32(np.max(np.abs(x[768:])))


def test_quantize8_rounds_half_to_even_and_handles_zero_block():
    a = 127.0
    x = np.array([a, 0.5, 1.5, 2.5, -0.5, -1.5])
    c, _ = O.quantize8(x, True)
    np.testing.assert_array_equal(c, np.array([127, 0, 2, 2, 0, -2], np.int8))
    c0, a0 = O.quantize8(np.zeros(300), False)
    assert not c0.any() and not a0.any()
    np.testing.assert_array_equal(O.dequantize8(c0, a0, False), np.zeros(300))


def test_round_bf16_matches_torch():
    x = np.concatenate([RNG.standard_normal(5000) * 10.0 ** RNG.integers(-20, 20, 5000),
                        np.array([0.0, 1.0, 1.00390625, 1.01171875, -3.0])])
    ref = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).double().numpy()
    np.testing.assert_array_equal(O.round_bf16(x), ref)


def test_precision_cosine_pins():
    o = O.Opts()
    m = RNG.standard_normal(2000) * 1e-3
    v = (RNG.standard_normal(2000) * 1e-3) ** 2 + 1e-8
    assert abs(O.precision_cosine(m, v, 32, o) - 1.0) < 1e-9
    q16, q8 = O.precision_cosine(m, v, 16, o), O.precision_cosine(m, v, 8, o)
    assert 0.0 < q8 <= q16 <= 1.0 + 1e-12 and q16 > 0.9999
    # exactly representable states: quantisation changes nothing, so Q(8) = 1
    a = np.float32(0.25)
    cm = RNG.integers(-127, 128, 512); cm[0] = 127; cm[256] = -127
    cv = RNG.integers(1, 256, 512); cv[0] = 255; cv[256] = 255
    mm = cm * float(a) / 127.0
    vv = cv * float(a) / 255.0
    assert abs(O.precision_cosine(mm, vv, 8, o) - 1.0) < 1e-9
    assert O.quant_rel_error(mm, 8, True, o) == 0.0 and O.quant_rel_error(vv, 8, False, o) == 0.0


def test_precision_cosine_explicit_small_case():
    # one quantisation block of 4: write Eq. 8 out by hand
    o = O.Opts(qblock=4, eps_adam=0.0, eps=0.0)
    m = np.array([1.0, -0.5, 0.26, 0.0])
    v = np.array([4.0, 1.0, 0.25, 2.0])
    mq = np.rint(127 * m / 1.0) / 127.0
    vq = np.rint(255 * v / 4.0) * 4.0 / 255.0
    u32, u8 = m / np.sqrt(v), mq / np.sqrt(vq)
    want = u32 @ u8 / (np.linalg.norm(u32) * np.linalg.norm(u8))
    assert abs(O.precision_cosine(m, v, 8, o) - want) < 1e-12


def test_precision_cosine_sixteen_bits_by_hand():
    """Eq. 8 at b = 16 on four elements whose bfloat16 neighbours are written out as literals (8 significant bits:
    a spacing of 2^-7 in [1, 2), 2^-9 in [1/4, 1/2), 2^-11 in [1/16, 1/8)), with two exact ties.  The value must
    also tell apart the mistakes that leave a moment un-rounded."""
    o = O.Opts(eps_adam=0.0, eps=0.0)
    m = np.array([1.00390625, -0.3, 1.01171875, 3.0])      # 1 + 2^-8: tie, to the even 1.0;  1 + 3*2^-8: tie, to 1 + 2^-6
    v = np.array([4.0, 0.1, 1.0078125, 2.0])               # 1 + 2^-7 is a bfloat16 already
    m16 = np.array([1.0, -0.30078125, 1.015625, 3.0])      # 0.3 = 1.2 * 2^-2 -> (1 + 26/128) / 4
    v16 = np.array([4.0, 0.10009765625, 1.0078125, 2.0])   # 0.1 = 1.6 * 2^-4 -> (1 + 77/128) / 16
    u32, u16 = m / np.sqrt(v), m16 / np.sqrt(v16)
    want = u32 @ u16 / (np.linalg.norm(u32) * np.linalg.norm(u16))
    got = O.precision_cosine(m, v, 16, o)
    assert abs(got - want) < 1e-14
    assert want < 1.0 - 1e-7                                # the rounding is visible in the value
    for mq, vq in ((m, v), (m16, v), (m, v16)):             # nothing rounded, only m, only v: all distinguishable
        ub = mq / np.sqrt(vq)
        wrong = u32 @ ub / (np.linalg.norm(u32) * np.linalg.norm(ub))
        assert abs(got - wrong) > 1e-8


def test_quant_rel_error_by_hand_at_eight_and_sixteen_bits():
    """||x - Q_b(x)|| / ||x|| on one quantisation block of four, every code and rounded value written out."""
    o = O.Opts(qblock=4)
    # signed 8-bit, absmax 1: 127 x = 127, -63.5 (tie, to the even 64), 33.02, 0
    x = np.array([1.0, -0.5, 0.26, 0.0])
    xq = np.array([127.0, -64.0, 33.0, 0.0]) / 127.0
    want = math.sqrt(float(np.sum((x - xq) ** 2))) / math.sqrt(1.0 + 0.25 + 0.26 ** 2)
    got = O.quant_rel_error(x, 8, True, o)
    assert want > 1e-3 and abs(got - want) < 1e-15
    assert abs(got - math.sqrt(float(np.sum((x - xq) ** 2))) / float(np.linalg.norm(xq))) > 1e-7   # not divided by ||Q(x)||
    # unsigned 8-bit, absmax 4: 255 v / 4 = 255, 63.75, 15.9375, 127.5 (tie, to the even 128)
    v = np.array([4.0, 1.0, 0.25, 2.0])
    vq = np.array([255.0, 64.0, 16.0, 128.0]) * 4.0 / 255.0
    want_v = math.sqrt(float(np.sum((v - vq) ** 2))) / math.sqrt(16.0 + 1.0 + 0.0625 + 4.0)
    assert want_v > 1e-3 and abs(O.quant_rel_error(v, 8, False, o) - want_v) < 1e-15
    # 16 bits: the bfloat16 literals of the test above (signedness does not enter)
    y = np.array([1.00390625, -0.3, 1.01171875, 0.1])
    yq = np.array([1.0, -0.30078125, 1.015625, 0.10009765625])
    want_y = math.sqrt(float(np.sum((y - yq) ** 2))) / math.sqrt(float(np.sum(y * y)))
    for signed in (True, False):
        assert abs(O.quant_rel_error(y, 16, signed, o) - want_y) < 1e-15
    assert want_y > 1e-3
    assert O.quant_rel_error(np.zeros(4), 8, True, o) == 0.0 and O.quant_rel_error(np.zeros(4), 16, True, o) == 0.0


def test_stats_finalize_reports_the_pinned_diagnostics():
    """The finalize record carries exactly the pinned functions' values (a wiring check: no swapped keys)."""
    o = O.Opts(qblock=4, eps_adam=0.0)
    st = O.stats_init(4)
    st.m = np.array([1.00390625, -0.3, 1.01171875, 0.1])
    st.v = np.array([4.0, 1.0, 0.25, 2.0])
    raw = O.stats_finalize(st, np.ones(4), 4, 1, o)
    assert raw["Q16"] == O.precision_cosine(st.m, st.v, 16, o) and raw["Q8"] == O.precision_cosine(st.m, st.v, 8, o)
    assert raw["err_m8"] == O.quant_rel_error(st.m, 8, True, o) and raw["err_v8"] == O.quant_rel_error(st.v, 8, False, o)
    assert raw["err_m16"] == O.quant_rel_error(st.m, 16, True, o) and raw["err_v16"] == O.quant_rel_error(st.v, 16, False, o)
    assert len({raw["err_m8"], raw["err_v8"], raw["err_m16"], raw["err_v16"]}) == 4


# ---------------------------------------------------------------- P6 normalisation (Eq. 10-20)

def _raw(**kw):
    base = dict(A=0.0, rho_bar=0.0, snr=0.0, C=0.0, F=0.0, Q32=1.0, Q16=1.0, Q8=1.0)
    base.update(kw)
    return base


def test_normalisation_anchor_values():
    o = O.Opts()
    z = O.normalise(_raw(A=math.log(2.0)), o); assert z["s_A"] == 0.0
    z = O.normalise(_raw(A=math.log(10.0)), o); assert abs(z["s_A"] - 1.0) < 1e-15
    z = O.normalise(_raw(A=0.5 * (math.log(2.0) + math.log(10.0))), o); assert abs(z["s_A"] - 0.5) < 1e-15
    z = O.normalise(_raw(A=5.0), o); assert z["s_A"] == 1.0
    z = O.normalise(_raw(A=-1.0), o); assert z["s_A"] == 0.0
    for rho, want in [(0.2, 0.0), (0.4, 0.5), (0.6, 1.0), (0.9, 1.0), (-0.5, 0.0)]:
        assert abs(O.normalise(_raw(rho_bar=rho), o)["s_rho"] - want) < 1e-15
    for s, want in [(0.0, 0.0), (math.e - 1.0, 0.5), (math.e ** 2 - 1.0, 1.0), (1e9, 1.0)]:
        assert abs(O.normalise(_raw(snr=s), o)["s_snr"] - want) < 1e-15
    z = O.normalise(_raw(rho_bar=0.4, snr=math.e - 1.0), o)
    assert abs(z["s_M"] - 0.25) < 1e-15
    assert abs(O.normalise(_raw(rho_bar=0.4, snr=math.e - 1.0), O.Opts(use_snr=False))["s_M"] - 0.5) < 1e-15
    assert abs(O.normalise(_raw(C=math.e - 1.0), o)["C_tilde"] - 1.0) < 1e-15
    assert O.normalise(_raw(F=1.7), o)["s_F"] == 1.0 and O.normalise(_raw(F=0.3), o)["s_F"] == 0.3
    z = O.normalise(_raw(Q8=0.5, Q16=-0.2, Q32=1.0), o)
    assert abs(z["lQ8"] - (-math.log(0.5 + 1e-12))) < 1e-15
    assert abs(z["lQ16"] - (-math.log(2e-12))) < 1e-12          # clipped to eps first (Eq. 10)
    assert abs(z["lQ32"] - (-math.log(1.0 + 1e-12))) < 1e-15


# ---------------------------------------------------------------- P7 risk and Agg (Eq. 1, Eq. 9)

def test_agg_of_the_five_configurations():
    assert [O.agg(c) for c in O.default_configs()] == [0.0, 3.0, 1.0, 2.0, 1.0]
    assert O.agg(O.Config(0, 0, 0, 1, 8)) == 7.0 and O.agg(O.Config(1, 1, 1, 0, 16)) == 1.0


def test_risk_is_linear_in_switches_with_distinct_terms():
    o = O.Opts(w=(2.0, 3.0, 5.0, 7.0, 11.0))
    z = dict(s_A=0.1, s_M=0.2, C_tilde=0.3, s_F=0.4, lQ32=0.0, lQ16=0.01, lQ8=0.05)
    assert abs(O.risk(z, O.Config(1, 1, 1, 0, 32), o)) < 1e-15
    assert abs(O.risk(z, O.Config(0, 1, 1, 0, 32), o) - 0.2) < 1e-15
    assert abs(O.risk(z, O.Config(1, 0, 1, 0, 32), o) - 0.6) < 1e-15
    assert abs(O.risk(z, O.Config(1, 1, 0, 0, 32), o) - 1.5) < 1e-15
    assert abs(O.risk(z, O.Config(1, 1, 1, 1, 32), o) - 2.8) < 1e-15
    assert abs(O.risk(z, O.Config(1, 1, 1, 0, 8), o) - 0.55) < 1e-15
    assert abs(O.risk(z, O.Config(0, 0, 0, 1, 16), o) - (0.2 + 0.6 + 1.5 + 2.8 + 0.11)) < 1e-12
    c = O.Config(1, 0, 1, 1, 32)
    assert abs(O.objective(1.0, c, O.Opts(), pref=0.25) - (0.75 + 0.1 * 2.0)) < 1e-15


# ---------------------------------------------------------------- P5 memory model

def test_state_bytes_model_and_paper_tables():
    cfg = O.default_configs()
    d, r, c = 1024 * 300, 1024, 300
    assert [O.state_bytes(k, d, r, c) for k in cfg] == [8 * d, 2 * d + 8 * (d // 256), 4 * d, 4 * (r + c), 4 * d]
    assert O.state_bytes(cfg[1], 257, 257, 1) == 2 * 257 + 8 * 2
    assert O.state_bytes(O.Config(1, 1, 1, 0, 16), d, r, c) == 4 * d
    g = _gold()
    per_param = 2.0 + 8.0 / 256.0
    for name in ("llama1b", "llama3b", "unet", "gpt2", "vit"):
        ratio = g[f"statemem_{name}_adamw8"] / g[f"statemem_{name}_adamw16"]
        # AdamW16 keeps 4 bytes of state per parameter; the tables' 8-bit rows then imply
        # 2 code bytes + two fp32 absmax per 256 elements (small tensors round up, hence the slack)
        assert abs(ratio * 4.0 - per_param) < 0.02, name
    assert abs(g["statemem_llama1b_adamw8"] / g["statemem_llama1b_adamw16"] * 4.0 - per_param) < 1e-3


# ---------------------------------------------------------------- P9 brute-force allocation (Eq. 2)

def test_bruteforce_hand_example_and_tie_break():
    phi = [[0, 5], [0, 5], [0, 5]]
    mem = [[4, 1], [4, 1], [4, 1]]
    r = [[1, 1]] * 3
    asg, val = O.allocate_bruteforce(phi, mem, r, 9, 100)
    assert asg == [0, 0, 1] and val == 5            # equal optima: lexicographically smallest wins
    asg, val = O.allocate_bruteforce(phi, mem, r, 12, 100)
    assert asg == [0, 0, 0] and val == 0
    asg, val = O.allocate_bruteforce(phi, mem, r, 2, 100)
    assert asg is None
    asg, val = O.allocate_bruteforce(phi, mem, [[3, 1]] * 3, 12, 5)   # time budget binds instead
    assert asg == [0, 1, 1] and val == 10
    asg, val = O.allocate_bruteforce(phi, mem, r, 12, 100, forbid=[[1, 0], [0, 0], [0, 0]])
    assert asg == [1, 0, 0]


def test_bruteforce_feasibility_and_monotonicity():
    rng = np.random.default_rng(5)
    for _ in range(20):
        n, k = 5, 3
        phi = rng.integers(0, 50, (n, k)).tolist()
        mem = rng.integers(1, 20, (n, k)).tolist()
        r = rng.integers(1, 10, (n, k)).tolist()
        prev = None
        for b in range(5, 100, 7):
            asg, val = O.allocate_bruteforce(phi, mem, r, b, 30)
            if asg is None:
                assert prev is None
                continue
            assert sum(mem[i][c] for i, c in enumerate(asg)) <= b
            assert sum(r[i][c] for i, c in enumerate(asg)) <= 30
            assert prev is None or val <= prev        # optimum never worsens as the budget grows
            prev = val


def test_fixed_point_helpers():
    assert O.phi_fixed(1.0) == 2 ** 30 and O.phi_fixed(-0.5) == -(2 ** 29)
    assert O.phi_fixed(1.5 / 2 ** 30) == 2 and O.phi_fixed(2.5 / 2 ** 30) == 2     # ties to even
    assert O.ratio_fixed(1.25) == 5 * 2 ** 18
    assert O.time_cap_fixed(3, 1.1) == math.floor(3 * 1.1 * 2 ** 20)


# ---------------------------------------------------------------- P10 update rules vs torch.optim (float64)

def _torch_run(opt_ctor, theta0, grads):
    p = torch.nn.Parameter(torch.from_numpy(theta0.copy()))
    opt = opt_ctor([p])
    for g in grads:
        p.grad = torch.from_numpy(g.copy())
        opt.step()
    return p.detach().numpy()


def _oracle_run(cfg, theta0, grads, rows, cols):
    st = O.step_init(cfg, theta0.shape[0], rows, cols)
    th = theta0.copy()
    for g in grads:
        th = O.step(th, g, st, cfg, rows, cols)
    return th, st


@pytest.mark.parametrize("wd,decoupled", [(0.0, 1), (0.05, 1), (0.05, 0)])
def test_fp32_adam_path_matches_torch(wd, decoupled):
    th0 = RNG.standard_normal(300)
    gs = [RNG.standard_normal(300) for _ in range(6)]
    cfg = O.Config(1, 1, decoupled, 0, 32, lr=3e-3, beta1=0.85, beta2=0.97, eps=1e-6, weight_decay=wd)
    if decoupled:
        ctor = lambda ps: torch.optim.AdamW(ps, lr=3e-3, betas=(0.85, 0.97), eps=1e-6, weight_decay=wd)
    else:
        ctor = lambda ps: torch.optim.Adam(ps, lr=3e-3, betas=(0.85, 0.97), eps=1e-6, weight_decay=wd)
    got, _ = _oracle_run(cfg, th0, gs, 300, 1)
    ref = _torch_run(ctor, th0, gs)
    # torch folds the bias corrections into the step size and the denominator; same value up to rounding
    np.testing.assert_allclose(got, ref, rtol=1e-10, atol=1e-13)


def test_sgd_momentum_path_matches_torch():
    th0 = RNG.standard_normal(200)
    gs = [RNG.standard_normal(200) for _ in range(5)]
    cfg = O.Config(0, 1, 0, 0, 32, lr=0.05, beta1=0.8, weight_decay=0.01)
    got, _ = _oracle_run(cfg, th0, gs, 200, 1)
    ref = _torch_run(lambda ps: torch.optim.SGD(ps, lr=0.05, momentum=0.8, weight_decay=0.01), th0, gs)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-14)
    # decoupled decay: theta shrinks by (1 - lr*wd) before the momentum step
    cfg2 = O.Config(0, 1, 1, 0, 32, lr=0.05, beta1=0.8, weight_decay=0.01)
    got2, _ = _oracle_run(cfg2, th0, gs[:1], 200, 1)
    np.testing.assert_allclose(got2, th0 * (1 - 0.05 * 0.01) - 0.05 * gs[0], rtol=1e-13)


def test_rms_path_is_adam_with_beta1_zero():
    th0 = RNG.standard_normal(128)
    gs = [RNG.standard_normal(128) for _ in range(5)]
    cfg = O.Config(1, 0, 1, 0, 32, lr=1e-3, beta2=0.99, eps=1e-7, weight_decay=0.02)
    got, st = _oracle_run(cfg, th0, gs, 128, 1)
    ref = _torch_run(lambda ps: torch.optim.AdamW(ps, lr=1e-3, betas=(0.0, 0.99), eps=1e-7, weight_decay=0.02), th0, gs)
    np.testing.assert_allclose(got, ref, rtol=1e-10, atol=1e-13)
    assert st.m is None                                   # no first moment is stored


# ---------------------------------------------------------------- P11 factored path

def test_factored_equals_rms_when_squares_are_rank_one():
    rows, cols = 24, 40
    th0 = RNG.standard_normal(rows * cols)
    x, y = RNG.random(rows) + 0.5, RNG.random(cols) + 0.5
    gs = []
    for _ in range(5):
        sign = RNG.choice([-1.0, 1.0], size=(rows, cols))
        gs.append((sign * np.outer(x, y)).reshape(-1))       # g^2 is the same rank-1 matrix each step
    f = O.Config(1, 0, 1, 1, 32, lr=2e-3, beta2=0.98, eps=1e-9, weight_decay=0.01)
    r = O.Config(1, 0, 1, 0, 32, lr=2e-3, beta2=0.98, eps=1e-9, weight_decay=0.01)
    a, st = _oracle_run(f, th0, gs, rows, cols)
    b, _ = _oracle_run(r, th0, gs, rows, cols)
    np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-13)
    assert st.r.shape == (rows,) and st.c.shape == (cols,)
    with pytest.raises(ValueError):
        O.step_init(f, 10, 10, 1)


def test_factored_hand_example():
    # one step, beta2 = 0: r = row means of g^2, c = column means, v = r c^T / mean(r)
    g = np.array([[1.0, 2.0], [3.0, 4.0]])
    cfg = O.Config(1, 0, 1, 1, 32, lr=1.0, beta2=0.0, eps=0.0, weight_decay=0.0)
    th, st = _oracle_run(cfg, np.zeros(4), [g.reshape(-1)], 2, 2)
    r = np.array([2.5, 12.5]); c = np.array([5.0, 10.0])
    v = np.outer(r, c) / 7.5
    np.testing.assert_allclose(st.r, r); np.testing.assert_allclose(st.c, c)
    np.testing.assert_allclose(th, (-g / np.sqrt(v)).reshape(-1), rtol=1e-13)


# ---------------------------------------------------------------- P12 8-bit path

def test_int8_path_zero_gradient_decay_and_lr_zero():
    n = 600
    a = np.float32(0.5)
    cfg = O.Config(1, 1, 1, 0, 8, lr=0.0, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
    st = O.step_init(cfg, n, n, 1)
    qm = RNG.integers(-127, 128, n); qm[0] = 127; qm[256] = 127; qm[512] = -127
    qv = RNG.integers(0, 256, n); qv[0] = 255; qv[256] = 255; qv[512] = 255
    st.qm, st.qv = qm.astype(np.int8), qv.astype(np.uint8)
    st.am = np.full(3, a, np.float32); st.av = np.full(3, a, np.float32)
    th0 = RNG.standard_normal(n)
    th = O.step(th0, np.zeros(n), st, cfg, n, 1)
    np.testing.assert_array_equal(th, th0)                           # lr = 0 leaves theta alone
    # m -> 0.9 m; the new absmax is 0.9 a (rounded to fp32), so the codes are unchanged
    np.testing.assert_array_equal(st.qm, qm.astype(np.int8))
    np.testing.assert_array_equal(st.qv, qv.astype(np.uint8))
    np.testing.assert_array_equal(st.am, np.full(3, np.float32(0.9 * float(a)), np.float32))
    np.testing.assert_array_equal(st.av, np.full(3, np.float32(0.999 * float(a)), np.float32))


def test_int8_path_tracks_fp32_path_within_one_code():
    n = 2048
    th0 = RNG.standard_normal(n) * 0.02
    gs = [RNG.standard_normal(n) * 1e-2 for _ in range(4)]
    c8 = O.Config(1, 1, 1, 0, 8, lr=1e-4, weight_decay=0.0)
    c32 = O.Config(1, 1, 1, 0, 32, lr=1e-4, weight_decay=0.0)
    # a single step from zero state: the 8-bit states are the quantised fp32 states exactly
    _, s8 = _oracle_run(c8, th0, gs[:1], n, 1)
    t32, s32 = _oracle_run(c32, th0, gs[:1], n, 1)
    t8, _ = _oracle_run(c8, th0, gs[:1], n, 1)
    np.testing.assert_allclose(t8, t32, rtol=1e-13)                  # theta uses un-requantised moments
    qm, am = O.quantize8(s32.m, True); qv, av = O.quantize8(s32.v, False)
    np.testing.assert_array_equal(s8.qm, qm); np.testing.assert_array_equal(s8.qv, qv)
    np.testing.assert_array_equal(s8.am, am); np.testing.assert_array_equal(s8.av, av)
    # second step: hand-computed from the dequantised state
    m1 = O.dequantize8(qm, am, True); v1 = O.dequantize8(qv, av, False)
    m2 = 0.9 * m1 + 0.1 * gs[1]; v2 = 0.999 * v1 + 0.001 * gs[1] ** 2
    th2 = t8 - 1e-4 * (m2 / (1 - 0.9 ** 2)) / (np.sqrt(v2 / (1 - 0.999 ** 2)) + 1e-8)
    got, s8b = _oracle_run(c8, th0, gs[:2], n, 1)
    np.testing.assert_allclose(got, th2, rtol=1e-12)
    q2, a2 = O.quantize8(m2, True)
    np.testing.assert_array_equal(s8b.qm, q2); np.testing.assert_array_equal(s8b.am, a2)


def test_config_kind_dispatch():
    kinds = [O.config_kind(c) for c in O.default_configs()]
    assert kinds == ["A32", "A8", "R", "F", "S"]
    assert O.config_kind(O.Config(0, 0, 1, 0, 32)) == "G" and O.config_kind(O.Config(0, 0, 0, 0, 8)) == "G"
    assert [O.config_kind(O.Config(1, 1, 1, 0, b)) for b in (32, 16, 8)] == ["A32", "A16", "A8"]
    assert [O.config_kind(O.Config(1, 0, 1, 0, b)) for b in (32, 16, 8)] == ["R", "R16", "R8"]
    assert [O.config_kind(O.Config(0, 1, 1, 0, b)) for b in (32, 16, 8)] == ["S", "S16", "S8"]
    assert [O.config_kind(O.Config(1, 0, 1, 1, b)) for b in (32, 16, 8)] == ["F", "F16", "F8"]
    assert O.config_kind(O.Config(1, 1, 1, 1, 32)) == "unsupported" and O.config_kind(O.Config(0, 0, 1, 1, 16)) == "unsupported"


def test_plain_gradient_step_matches_torch_sgd():
    rng = np.random.default_rng(7)
    th0 = rng.standard_normal(37)
    for decoupled, wd in ((1, 0.0), (0, 0.1)):
        c = O.Config(0, 0, decoupled, 0, 32, lr=0.05, weight_decay=wd)
        st = O.step_init(c, 37, 37, 1)
        p = torch.tensor(th0, dtype=torch.float64, requires_grad=True)
        opt = torch.optim.SGD([p], lr=0.05, momentum=0.0, weight_decay=wd)     # torch's decay is the coupled one
        th = th0.copy()
        for t in range(4):
            g = rng.standard_normal(37)
            th = O.step(th, g, st, c, 37, 1)
            p.grad = torch.tensor(g, dtype=torch.float64)
            opt.step()
        np.testing.assert_allclose(th, p.detach().numpy(), rtol=1e-13, atol=1e-15)
    # decoupled decay: theta (1 - lr wd) - lr g, by hand
    c = O.Config(0, 0, 1, 0, 32, lr=0.5, weight_decay=0.2)
    np.testing.assert_allclose(O.step(np.array([2.0]), np.array([1.0]), O.step_init(c, 1, 1, 1), c, 1, 1), [2.0 * 0.9 - 0.5])
    assert O.state_bytes(c, 100, 100, 1) == 0


def test_bf16_state_rules_store_rounded_moments_and_update_with_unrounded_ones():
    rng = np.random.default_rng(11)
    n = 300
    g_seq = [O.round_bf16(rng.standard_normal(n) * 0.01) for _ in range(5)]
    for full, half in ((O.Config(1, 1, 1, 0, 32, weight_decay=0.01), O.Config(1, 1, 1, 0, 16, weight_decay=0.01)),
                       (O.Config(1, 0, 1, 0, 32), O.Config(1, 0, 1, 0, 16)),
                       (O.Config(0, 1, 0, 0, 32, lr=1e-2, weight_decay=0.1), O.Config(0, 1, 0, 0, 16, lr=1e-2, weight_decay=0.1))):
        s32, s16 = O.step_init(full, n, n, 1), O.step_init(half, n, n, 1)
        th32 = th16 = rng.standard_normal(n) * 0.02
        # first step from the zero state: same update (the un-rounded moments are used), stored moments are the bf16
        # roundings of the fp32-path moments
        th32 = O.step(th32, g_seq[0], s32, full, n, 1)
        th16 = O.step(th16, g_seq[0], s16, half, n, 1)
        np.testing.assert_array_equal(th32, th16)
        for name in ("m", "v"):
            a32, a16 = getattr(s32, name), getattr(s16, name)
            if a32 is not None:
                np.testing.assert_array_equal(a16, O.round_bf16(a32))
                assert np.all(np.abs(a16 - a32) <= np.abs(a32) * 2.0 ** -8)           # half a bf16 spacing at most
        # later steps start from the rounded state: stays within bf16 resolution of the fp32 path, but differs
        for g in g_seq[1:]:
            th32 = O.step(th32, g, s32, full, n, 1)
            th16 = O.step(th16, g, s16, half, n, 1)
        assert 0 < np.max(np.abs(th32 - th16)) < 1e-2 * np.max(np.abs(th32))
        for name in ("m", "v"):
            a16 = getattr(s16, name)
            if a16 is not None:
                np.testing.assert_array_equal(a16, O.round_bf16(a16))                     # the state is always bf16
    assert O.state_bytes(O.Config(1, 1, 1, 0, 16), 1000, 1000, 1) == 4000
    assert O.state_bytes(O.Config(0, 1, 1, 0, 16), 1000, 1000, 1) == 2000


def test_int8_single_moment_rules_follow_their_fp32_forms():
    rng = np.random.default_rng(13)
    n = 700                                                       # three quantisation blocks, the last one ragged
    g0 = O.round_bf16(rng.standard_normal(n) * 0.01)
    th0 = rng.standard_normal(n) * 0.02
    for full, q, name, signed in ((O.Config(1, 0, 1, 0, 32), O.Config(1, 0, 1, 0, 8), "v", False),
                                  (O.Config(0, 1, 0, 0, 32, lr=1e-2, weight_decay=0.1), O.Config(0, 1, 0, 0, 8, lr=1e-2, weight_decay=0.1), "m", True)):
        s32, s8 = O.step_init(full, n, n, 1), O.step_init(q, n, n, 1)
        a = O.step(th0, g0, s32, full, n, 1)
        b = O.step(th0, g0, s8, q, n, 1)
        np.testing.assert_array_equal(a, b)                       # from the zero state the un-requantised moment is the fp32 one
        codes, absmax = O.quantize8(getattr(s32, name), signed)
        np.testing.assert_array_equal(getattr(s8, "q" + name), codes)
        np.testing.assert_array_equal(getattr(s8, "a" + name), absmax)
        # zero gradient, no decay: the state only decays; the codes move by rne(beta * code) up to the new absmax
        z = O.Config(q.adaptive, q.momentum, 1, 0, 8, lr=0.0, beta1=0.5, beta2=0.5)
        before = getattr(s8, "q" + name).astype(np.int32).copy()
        th = O.step(b, np.zeros(n), s8, z, n, 1)
        np.testing.assert_array_equal(th, b)                      # lr = 0: parameters unchanged
        after = getattr(s8, "q" + name).astype(np.int32)
        assert np.all(np.abs(after - before) <= 1)                # rescaling by the decayed absmax keeps the codes
    assert O.state_bytes(O.Config(1, 0, 1, 0, 8), 700, 700, 1) == 700 + 4 * 3
    assert O.state_bytes(O.Config(0, 1, 1, 0, 8), 700, 700, 1) == 700 + 4 * 3


def test_reconfigure_inherits_compatible_moments_and_restarts_the_rest():
    rng = np.random.default_rng(17)
    rows, cols = 24, 32
    n = rows * cols
    a32 = O.Config(1, 1, 1, 0, 32)
    st = O.step_init(a32, n, rows, cols)
    th = rng.standard_normal(n) * 0.02
    for _ in range(3):
        th = O.step(th, O.round_bf16(rng.standard_normal(n) * 0.01), st, a32, rows, cols)
    m, v = st.m.copy(), st.v.copy()
    # same tuple: nothing changes but the storage rounding to fp32
    same = O.reconfigure(st, a32, rows, cols)
    np.testing.assert_array_equal(same.m, m.astype(np.float32).astype(np.float64))
    assert (same.t, same.t_m0, same.t_v0) == (3, 0, 0)
    # Adam fp32 -> 8-bit: the codes are the quantisation of the moments; -> bf16: their rounding
    a8 = O.reconfigure(st, O.Config(1, 1, 1, 0, 8), rows, cols)
    q, a = O.quantize8(m, True)
    np.testing.assert_array_equal(a8.qm, q); np.testing.assert_array_equal(a8.am, a)
    q, a = O.quantize8(v, False)
    np.testing.assert_array_equal(a8.qv, q); np.testing.assert_array_equal(a8.av, a)
    a16 = O.reconfigure(st, O.Config(1, 1, 1, 0, 16), rows, cols)
    np.testing.assert_array_equal(a16.v, O.round_bf16(v))
    # 8-bit -> fp32: the dequantised values, within half a code of the originals
    back = O.reconfigure(a8, a32, rows, cols)
    assert np.max(np.abs(back.m - m)) <= np.max(np.abs(m)) / 254 * 1.0001 and (back.t_m0, back.t_v0) == (0, 0)
    # Adam -> RMS keeps v and drops m; Adam -> SGD-momentum keeps nothing (another family) and restarts the buffer
    r = O.reconfigure(st, O.Config(1, 0, 1, 0, 32), rows, cols)
    np.testing.assert_array_equal(r.v, v.astype(np.float32).astype(np.float64)); assert r.m is None and r.t_v0 == 0
    s = O.reconfigure(st, O.Config(0, 1, 1, 0, 32), rows, cols)
    assert not s.m.any() and s.t_m0 == 3
    # RMS -> Adam: v continues with its age, m starts from zero with a fresh bias correction
    back2 = O.reconfigure(r, a32, rows, cols)
    assert not back2.m.any() and (back2.t_m0, back2.t_v0) == (3, 0)
    g = O.round_bf16(rng.standard_normal(n) * 0.01)
    th2 = O.step(th, g, back2, a32, rows, cols)                      # step 4: m has seen 1 gradient, v has seen 4
    m1 = (1 - a32.beta1) * g
    v4 = a32.beta2 * r.v + (1 - a32.beta2) * g * g
    want = th * (1 - a32.lr * a32.weight_decay) - a32.lr * (m1 / (1 - a32.beta1)) / (np.sqrt(v4 / (1 - a32.beta2 ** 4)) + a32.eps)
    np.testing.assert_allclose(th2, want, rtol=1e-12, atol=1e-15)
    # element-wise -> factored: row and column means; factored -> element-wise: r_i c_j / mean(r)
    f = O.reconfigure(st, O.Config(1, 0, 1, 1, 32), rows, cols)
    V = v.reshape(rows, cols)
    np.testing.assert_allclose(f.r, V.mean(axis=1), rtol=1e-7); np.testing.assert_allclose(f.c, V.mean(axis=0), rtol=1e-7)
    full = O.reconfigure(f, O.Config(1, 0, 1, 0, 32), rows, cols)
    np.testing.assert_allclose(full.v, (np.outer(f.r, f.c) / f.r.mean()).reshape(-1), rtol=1e-7)
    # without inheritance everything restarts
    z = O.reconfigure(st, O.Config(1, 1, 1, 0, 32), rows, cols, inherit=False)
    assert not z.m.any() and not z.v.any() and (z.t_m0, z.t_v0) == (3, 3)


def test_warm_start_equals_training_that_held_the_parameters_still_during_the_window():
    """Carrying the window's moments into training must give what the optimizer itself would hold had it run through
    the window with a zero learning rate: same moments, same ages in the bias corrections."""
    import dataclasses
    rng = np.random.default_rng(23)
    rows, cols, T_w = 12, 32, 4
    n = rows * cols
    o = O.Opts()
    win = O.stats_init(n)
    gs = [O.round_bf16(rng.standard_normal(n) * 0.01) for _ in range(T_w + 2)]
    for g in gs[:T_w]:
        O.stats_step(win, g, o)
    th0 = rng.standard_normal(n) * 0.02
    for c in (O.Config(1, 1, 1, 0, 32), O.Config(1, 0, 0, 0, 32), O.Config(0, 1, 1, 0, 32, lr=1e-2), O.Config(1, 0, 1, 1, 32)):
        still = dataclasses.replace(c, lr=0.0, weight_decay=0.0)
        ref = O.step_init(c, n, rows, cols)
        th_ref = th0.copy()
        for g in gs[:T_w]:
            th_ref = O.step(th_ref, g, ref, still, rows, cols)
        np.testing.assert_array_equal(th_ref, th0)
        ws = O.warm_start(win, c, rows, cols, o)
        assert ws.t == 0
        if ws.m is not None:
            np.testing.assert_allclose(ws.m, ref.m, rtol=1e-7, atol=1e-30)
            assert ws.t_m0 == -T_w
        if ws.v is not None:
            np.testing.assert_allclose(ws.v, ref.v, rtol=1e-7, atol=1e-30)
        if ws.r is not None:
            # the factored statistics of the window's v_hat are the EMAs of the row and column means of g^2
            np.testing.assert_allclose(ws.r, ref.r, rtol=1e-6); np.testing.assert_allclose(ws.c, ref.c, rtol=1e-6)
        th_ws = th0.copy()
        for g in gs[T_w:]:
            th_ref = O.step(th_ref, g, ref, c, rows, cols)
            th_ws = O.step(th_ws, g, ws, c, rows, cols)
        np.testing.assert_allclose(th_ws, th_ref, rtol=2e-6, atol=1e-12)
    # a coefficient that differs from the window's: that moment starts from zero with a fresh bias correction
    c = O.Config(1, 1, 1, 0, 32, beta1=0.8)
    ws = O.warm_start(win, c, rows, cols, o)
    assert not ws.m.any() and (ws.t_m0, ws.t_v0) == (0, -T_w)
    np.testing.assert_array_equal(ws.v, win.v.astype(np.float32).astype(np.float64))
    # 8-bit and bf16 tuples store the window's moments in their own precision
    a8 = O.warm_start(win, O.Config(1, 1, 1, 0, 8), rows, cols, o)
    q, a = O.quantize8(win.m, True)
    np.testing.assert_array_equal(a8.qm, q); np.testing.assert_array_equal(a8.am, a)
    s16 = O.warm_start(win, O.Config(0, 1, 1, 0, 16), rows, cols, o)
    np.testing.assert_array_equal(s16.m, O.round_bf16(win.m / (1.0 - o.beta_m)))
    # the plain gradient step has nothing to carry
    assert O.warm_start(win, O.Config(0, 0, 1, 0, 32), rows, cols, o).m is None


def test_factored_states_in_reduced_precision():
    """Factored second moment with bf16 / 8-bit row and column statistics: the first step equals the fp32 one (the
    update uses the new statistics before they are rounded), what is stored is the rounding / the codes of them, the
    next step starts from the stored values, and the trajectories stay within the storage error of the fp32 one."""
    rng = np.random.default_rng(29)
    rows, cols = 300, 70                                   # more than one quantisation block of rows, a ragged one
    n = rows * cols
    f32, f16, f8 = (O.Config(1, 0, 1, 1, b) for b in (32, 16, 8))
    assert O.state_bytes(f32, n, rows, cols) == 4 * (rows + cols)
    assert O.state_bytes(f16, n, rows, cols) == 2 * (rows + cols)
    assert O.state_bytes(f8, n, rows, cols) == rows + cols + 4 * (2 + 1)
    th0 = rng.standard_normal(n) * 0.02
    g1 = O.round_bf16(rng.standard_normal(n) * 0.01 * (1 + np.arange(n) % 7))
    sts = {k: O.step_init(c, n, rows, cols) for k, c in (("F", f32), ("F16", f16), ("F8", f8))}
    out = {k: O.step(th0, g1, sts[k], c, rows, cols) for k, c in (("F", f32), ("F16", f16), ("F8", f8))}
    np.testing.assert_array_equal(out["F16"], out["F"])
    np.testing.assert_array_equal(out["F8"], out["F"])
    np.testing.assert_array_equal(sts["F16"].r, O.round_bf16(sts["F"].r))
    q, a = O.quantize8(sts["F"].c, False)
    np.testing.assert_array_equal(sts["F8"].qc, q); np.testing.assert_array_equal(sts["F8"].ac, a)
    assert sts["F8"].ar.shape == (2,) and sts["F8"].ac.shape == (1,)
    # second step by hand from the stored bf16 values
    g2 = O.round_bf16(rng.standard_normal(n) * 0.01)
    r_old, c_old = sts["F16"].r.copy(), sts["F16"].c.copy()
    th2 = O.step(out["F16"], g2, sts["F16"], f16, rows, cols)
    G2 = (g2 * g2).reshape(rows, cols)
    r = f16.beta2 * r_old + (1 - f16.beta2) * G2.mean(axis=1)
    c = f16.beta2 * c_old + (1 - f16.beta2) * G2.mean(axis=0)
    v = (np.outer(r, c) / r.mean()).reshape(-1)
    want = out["F16"] * (1 - f16.lr * f16.weight_decay) - f16.lr * g2 / (np.sqrt(v / (1 - f16.beta2 ** 2)) + f16.eps)
    np.testing.assert_allclose(th2, want, rtol=1e-13, atol=1e-16)
    np.testing.assert_array_equal(sts["F16"].r, O.round_bf16(r))
    # a few more steps: the reduced-precision runs track the fp32 one within the storage error of sqrt(v)
    th = {k: out[k] for k in out}
    th["F16"] = th2
    th["F"] = O.step(th["F"], g2, sts["F"], f32, rows, cols)
    th["F8"] = O.step(th["F8"], g2, sts["F8"], f8, rows, cols)
    for _ in range(4):
        g = O.round_bf16(rng.standard_normal(n) * 0.01)
        for k, c_ in (("F", f32), ("F16", f16), ("F8", f8)):
            th[k] = O.step(th[k], g, sts[k], c_, rows, cols)
    moved = np.max(np.abs(th["F"] - th0))
    assert np.max(np.abs(th["F16"] - th["F"])) <= 0.01 * moved
    assert np.max(np.abs(th["F8"] - th["F"])) <= 0.05 * moved
    assert np.max(np.abs(th["F8"] - th["F"])) > 0
    # migration between the precisions: decode, then store in the new form
    back = O.reconfigure(sts["F8"], f32, rows, cols)
    np.testing.assert_array_equal(back.r, O.dequantize8(sts["F8"].qr, sts["F8"].ar, False).astype(np.float32).astype(np.float64))
    down = O.reconfigure(sts["F"], f8, rows, cols)
    q, a = O.quantize8(sts["F"].r, False)
    np.testing.assert_array_equal(down.qr, q); np.testing.assert_array_equal(down.ar, a)
    full = O.reconfigure(sts["F16"], O.Config(1, 0, 1, 0, 32), rows, cols)
    np.testing.assert_allclose(full.v, (np.outer(sts["F16"].r, sts["F16"].c) / sts["F16"].r.mean()).reshape(-1), rtol=1e-7)


# ---------------------------------------------------------------- block partitioning (Algorithm 2)

def test_partition_threshold_is_the_upper_quartile_of_pairwise_differences():
    Z = np.array([[0.0], [1.0], [3.0]])
    ids, tau = O.partition_blocks([10, 10, 10], Z)
    assert tau == 2.5                                       # differences 1, 2, 3: position 0.75 * 2 = 1.5
    Zr = RNG.random((9, 5))
    w = np.array([1.0, 2.0, 0.5, 1.0, 3.0])
    pair = [np.max(w * np.abs(Zr[a] - Zr[b])) for a in range(9) for b in range(a + 1, 9)]
    assert abs(O.partition_blocks([5] * 9, Zr, w)[1] - np.quantile(pair, 0.75)) < 1e-15
    assert O.partition_delta(np.array([0.0, 1.0]), np.array([0.5, 0.0]), np.array([4.0, 1.0])) == 2.0


def test_partition_identical_units_form_one_block_and_clusters_split_at_their_edge():
    ids, tau = O.partition_blocks([7] * 6, np.full((6, 3), 0.4))
    assert tau == 0.0 and ids.tolist() == [0] * 6
    Z = np.array([[0.1, 0.2]] * 3 + [[0.9, 0.2]] * 4 + [[0.9, 0.8]] * 2)
    ids, _ = O.partition_blocks([10] * 9, Z, tau=0.5)
    assert ids.tolist() == [0, 0, 0, 1, 1, 1, 1, 2, 2]
    # the weights enter the difference: with the first diagnostic switched off only the second edge remains
    ids, _ = O.partition_blocks([10] * 9, Z, w=[0.0, 1.0], tau=0.5)
    assert ids.tolist() == [0] * 7 + [1, 1]


def test_partition_small_units_join_their_statistically_closest_neighbour():
    Z = np.array([[0.0], [0.9], [1.0]])
    ids, _ = O.partition_blocks([100, 1, 100], Z, alpha=5 / 201, tau=0.5)
    assert ids.tolist() == [0, 1, 1]
    ids, _ = O.partition_blocks([100, 1, 100], np.array([[0.0], [0.1], [1.0]]), alpha=5 / 201, tau=0.5)
    assert ids.tolist() == [0, 0, 1]
    # equal differences: the smaller neighbour takes it
    ids, _ = O.partition_blocks([100, 1, 50], np.array([[0.0], [0.5], [1.0]]), alpha=5 / 151, tau=0.3)
    assert ids.tolist() == [0, 1, 1]
    # a unit below the minimum never stays alone, whatever its statistics
    ids, _ = O.partition_blocks([50, 2, 50, 3], np.array([[0.0], [9.0], [0.0], [-9.0]]), alpha=0.05, tau=0.1)
    sizes = np.bincount(ids, weights=[50, 2, 50, 3])
    assert np.all(sizes >= 0.05 * 105)


def test_partition_splits_a_chain_of_small_steps_where_its_sides_differ():
    # adjacent differences 0.3, 0.6, 0.3 <= tau, so block formation merges everything; the means of the two sides
    # differ by 0.8, 0.9, 0.8 at the three cuts: the middle one wins and exceeds tau, the halves stay whole (0.3)
    Z = np.array([[0.0], [0.3], [0.9], [1.2]])
    ids, _ = O.partition_blocks([10] * 4, Z, tau=0.7)
    assert ids.tolist() == [0, 0, 1, 1]
    # the cut respects the minimum size: with n_min = 25 neither side of the middle cut fits
    ids, _ = O.partition_blocks([10] * 4, Z, alpha=15 / 40, tau=0.7)
    assert ids.tolist() == [0, 0, 1, 1]
    ids, _ = O.partition_blocks([10] * 4, Z, alpha=25 / 40, tau=0.7)
    assert ids.tolist() == [0, 0, 0, 0]
    # weighted means: the heavy third unit pulls its side to 0.9, so the cut after the first unit separates most
    # (0 against 0.897; the middle cut gives 0.15 against 0.903), and the rest holds together (0.3 against 0.903)
    ids, _ = O.partition_blocks([10, 10, 1000, 10], Z, tau=0.7)
    assert ids.tolist() == [0, 1, 1, 1]


def test_partition_invariants_on_random_inputs():
    rng = np.random.default_rng(5)
    for trial in range(40):
        m = int(rng.integers(1, 30))
        sizes = rng.integers(1, 1000, size=m).tolist()
        Z = rng.random((m, 5))
        alpha = float(rng.choice([0.0, 0.01, 0.05, 0.2]))
        ids, tau = O.partition_blocks(sizes, Z, alpha=alpha)
        assert ids[0] == 0 and np.all(np.diff(ids) >= 0) and np.all(np.diff(ids) <= 1)     # contiguous, in order
        per = np.bincount(ids, weights=sizes)
        assert len(per) == 1 or np.all(per >= alpha * sum(sizes))
        # a boundary that survived separates blocks whose statistics differ by more than tau, or was forced by nothing:
        # merging two adjacent final blocks must not be something block formation would have done
        if alpha == 0.0:
            for b in range(len(per) - 1):
                za = O._mean_z(sizes, Z, np.nonzero(ids == b)[0]); zb = O._mean_z(sizes, Z, np.nonzero(ids == b + 1)[0])
                members_a, members_b = np.nonzero(ids == b)[0], np.nonzero(ids == b + 1)[0]
                edge = O.partition_delta(Z[members_a[-1]], Z[members_b[0]], np.ones(5))
                assert edge > tau or O.partition_delta(za, zb, np.ones(5)) > tau


# ---------------------------------------------------------------- non-linear 8-bit codebook (alternative reading of the quantiser)

def test_dynamic_codebook_entries_by_hand():
    ts, tu = O.dynamic_codebook(True), O.dynamic_codebook(False)
    assert ts.shape == (255,) and tu.shape == (256,)
    assert np.all(np.diff(ts) > 0) and np.all(np.diff(tu) > 0)
    np.testing.assert_array_equal(ts, -ts[::-1])                     # symmetric; the middle entry is zero
    assert ts[127] == 0.0 and tu[0] == 0.0 and ts[-1] == 1.0 and ts[0] == -1.0 and tu[-1] == 1.0
    # decade E of the signed type has 2^(6-E) entries in (10^-(E+1), 10^-E]; written out: the top decade 64 steps of
    # 0.9/64 above 0.1, the next one 32 steps of 0.09/32 above 0.01, ..., the last one the single value 1e-6
    pos = ts[128:]
    assert pos.shape == (127,)
    assert abs(pos[0] - 1e-6) < 1e-21 and abs(pos[1] - 0.55e-5) < 1e-20 and abs(pos[2] - 1e-5) < 1e-20
    assert abs(pos[-64] - (0.1 + 0.9 / 64)) < 1e-16 and abs(pos[-65] - 0.1) < 1e-16 and abs(pos[-2] - (1.0 - 0.9 / 64)) < 1e-16
    for E in range(7):
        n = int(np.sum((pos > 10.0 ** -(E + 1) * (1 + 1e-12)) & (pos <= 10.0 ** -E * (1 + 1e-12))))
        assert n == 2 ** (6 - E), (E, n)
    # unsigned: one more fraction bit per decade and one more decade
    upos = tu[1:]
    assert abs(upos[0] - 1e-7) < 1e-22 and abs(upos[-128] - (0.1 + 0.9 / 128)) < 1e-16
    for E in range(8):
        assert int(np.sum((upos > 10.0 ** -(E + 1) * (1 + 1e-12)) & (upos <= 10.0 ** -E * (1 + 1e-12)))) == 2 ** (7 - E)


def test_dynamic_codebook_round_trip_nearest_entry_and_ties():
    for signed in (True, False):
        t = O.dynamic_codebook(signed)
        a = np.float32(0.5)                                           # a power of two: entry * a is exact
        x = t * float(a)
        if not signed:
            x = x.copy()                                              # the block's absmax must be a: its last entry is 1 * a
        codes, am = O.quantize8_dynamic(x, signed, qblock=len(t))
        np.testing.assert_array_equal(codes, np.arange(len(t), dtype=np.uint8))
        assert am.tolist() == [0.5]
        np.testing.assert_array_equal(O.dequantize8_dynamic(codes, am, signed, qblock=len(t)), x)
        # nearest entry: brute force over the table
        y = RNG.uniform(-1.0 if signed else 0.0, 1.0, 3000)
        y[0] = 1.0                                                    # absmax 1
        codes, am = O.quantize8_dynamic(y, signed, qblock=3000)
        brute = np.argmin(np.abs(y[:, None] - t[None, :]), axis=1)
        np.testing.assert_array_equal(codes, brute.astype(np.uint8))
        # a tie goes to the entry of smaller magnitude
        k = len(t) - 3
        tie = np.array([1.0, 0.5 * (t[k] + t[k + 1])])
        assert O.quantize8_dynamic(tie, signed, qblock=2)[0][1] == k
    ts = O.dynamic_codebook(True)
    tie = np.array([-1.0, 0.5 * (ts[2] + ts[3])])
    assert O.quantize8_dynamic(tie, True, qblock=2)[0][1] == 3        # negative: the upper entry is the smaller one
    c0, a0 = O.quantize8_dynamic(np.zeros(300), True)
    assert not a0.any() and not O.dequantize8_dynamic(c0, a0, True).any()


def test_dynamic_codebook_keeps_small_second_moments_that_linear_codes_lose():
    """What the non-linear table is for: a second moment 1e-4 of its block's absmax survives (relative error below 10 %)
    where the linear code rounds it to zero."""
    v = np.array([1.0, 1e-4, 3e-6, 0.0])
    cl, al = O.quantize8(v, False, 4)
    assert O.dequantize8(cl, al, False, 4)[1] == 0.0
    cd, ad = O.quantize8_dynamic(v, False, 4)
    vd = O.dequantize8_dynamic(cd, ad, False, 4)
    assert abs(vd[1] - 1e-4) <= 0.1 * 1e-4 and abs(vd[2] - 3e-6) <= 0.2 * 3e-6 and vd[3] == 0.0 and vd[0] == 1.0


def test_adam_on_the_dynamic_codebook_by_hand_and_against_fp32():
    c = O.Config(1, 1, 1, 0, 8, lr=1e-2, beta1=0.5, beta2=0.5, eps=0.0, weight_decay=0.0, quantizer="dynamic")
    assert O.config_kind(c) == "A8N"
    st = O.step_init(c, 2, 2, 1, qblock=2)
    g = np.array([1.0, -0.25])
    th = O.step(np.zeros(2), g, st, c, 2, 1, qblock=2)
    # m = g/2, v = g^2/2; bias corrections 1/2 each: theta = -lr * g / |g|
    np.testing.assert_allclose(th, [-1e-2, 1e-2], rtol=0, atol=1e-15)
    ts, tu = O.dynamic_codebook(True), O.dynamic_codebook(False)
    assert st.am.tolist() == [0.5] and st.av.tolist() == [0.5]
    # m / a = (1, -0.25): 0.25 lies between the entries 0.1 + 0.9 * 10/64 = 0.240625 and 0.1 + 0.9 * 11/64 = 0.2546875
    assert ts[st.qm[0]] == 1.0 and abs(ts[st.qm[1]] + 0.2546875) < 1e-16
    # v / a = (1, 1/16): the decade (0.01, 0.1] of the unsigned type has 64 entries 0.01 + 0.09 (k+1)/64; k + 1 = 37 is nearest
    assert tu[st.qv[0]] == 1.0 and abs(tu[st.qv[1]] - (0.01 + 0.09 * 37 / 64)) < 1e-16
    # ten steps stay close to the fp32 rule (the codebook's relative error is a few per cent per entry)
    c32 = O.Config(1, 1, 1, 0, 32, lr=1e-3, weight_decay=0.01)
    c8n = O.Config(1, 1, 1, 0, 8, lr=1e-3, weight_decay=0.01, quantizer="dynamic")
    d = 700
    s32, s8 = O.step_init(c32, d, d, 1), O.step_init(c8n, d, d, 1)
    th32 = th8 = RNG.standard_normal(d) * 0.02
    for t in range(10):
        g = RNG.standard_normal(d) * 1e-2
        th32, th8 = O.step(th32, g, s32, c32, d, 1), O.step(th8, g, s8, c8n, d, 1)
    assert np.max(np.abs(th32 - th8)) < 5e-4 and np.max(np.abs(th32 - th8)) > 0.0
    m8 = O.dequantize8_dynamic(s8.qm, s8.am, True)
    assert np.max(np.abs(m8 - s32.m)) <= 0.08 * np.max(np.abs(s32.m))


def test_precision_cosine_with_the_dynamic_codebook():
    o = O.Opts(qblock=4, eps_adam=0.0, eps=0.0, quantizer8="dynamic")
    m = np.array([1.0, -0.5, 0.26, 0.0])
    v = np.array([4.0, 1.0, 0.25, 2.0])
    ts, tu = O.dynamic_codebook(True), O.dynamic_codebook(False)
    near = lambda t, y: t[np.argmin(np.abs(t - y))]
    mq = np.array([near(ts, x / 1.0) * 1.0 for x in m])
    vq = np.array([near(tu, x / 4.0) * 4.0 for x in v])
    u32, u8 = m / np.sqrt(v), mq / np.sqrt(vq)
    want = u32 @ u8 / (np.linalg.norm(u32) * np.linalg.norm(u8))
    assert abs(O.precision_cosine(m, v, 8, o) - want) < 1e-14
    assert abs(O.precision_cosine(m, v, 8, o) - O.precision_cosine(m, v, 8, O.Opts(qblock=4, eps_adam=0.0, eps=0.0))) > 1e-9
    want_err = math.sqrt(float(np.sum((v - vq) ** 2))) / math.sqrt(float(np.sum(v * v)))
    assert abs(O.quant_rel_error(v, 8, False, o) - want_err) < 1e-15


# ---------------------------------------------------------------- Adafactor options of the factored tuple

def test_adafactor_options_off_is_the_mechanism_pure_rule():
    G = RNG.standard_normal((5, 7))
    th0 = RNG.standard_normal(35) * 0.02
    base = O.Config(1, 0, 1, 1, 32, lr=1e-3, beta2=0.9, weight_decay=0.01)
    same = O.Config(1, 0, 1, 1, 32, lr=1e-3, beta2=0.9, weight_decay=0.01, af_beta2_schedule=False, af_clip=0.0,
                    af_relative_step=False, af_eps1=0.0)
    s1, s2 = O.step_init(base, 35, 5, 7), O.step_init(same, 35, 5, 7)
    np.testing.assert_array_equal(O.step(th0, G.reshape(-1), s1, base, 5, 7), O.step(th0, G.reshape(-1), s2, same, 5, 7))


def test_adafactor_beta2_schedule_clipping_and_relative_step_by_hand():
    # a 2 x 2 block, two steps, every quantity written out
    G1 = np.array([[3.0, 1.0], [1.0, 2.0]])
    G2 = np.array([[1.0, -2.0], [0.5, 1.0]])
    th0 = np.array([0.5, -0.5, 0.25, 1.0])
    c = O.Config(1, 0, 1, 1, 32, lr=123.0, beta2=0.999, eps=0.0, weight_decay=0.0, af_beta2_schedule=True, af_clip=1.0,
                 af_relative_step=True, af_eps1=1e-30)
    st = O.step_init(c, 4, 2, 2)
    th1 = O.step(th0, G1.reshape(-1), st, c, 2, 2)
    # step 1: beta2_1 = 1 - 1^-0.8 = 0, so r and c are the row and column means of g^2 (+ eps1, invisible here)
    r1, c1 = np.array([5.0, 2.5]), np.array([5.0, 2.5])
    np.testing.assert_allclose(st.r, r1, rtol=1e-15); np.testing.assert_allclose(st.c, c1, rtol=1e-15)
    v1 = np.outer(r1, c1) / 3.75
    u1 = G1 / np.sqrt(v1)                                             # no bias correction under the schedule
    rms1 = math.sqrt(float(np.mean(u1 ** 2)))
    assert rms1 > 1.0
    u1 = u1 / rms1                                                    # clipped to RMS 1 (d = 1)
    alpha1 = max(1e-3, math.sqrt(float(np.mean(th0 ** 2)))) * min(1e-2, 1.0)
    np.testing.assert_allclose(th1, th0 - alpha1 * u1.reshape(-1), rtol=1e-14)
    th2 = O.step(th1, G2.reshape(-1), st, c, 2, 2)
    b2 = 1.0 - 2.0 ** -0.8                                            # 0.42565...
    assert abs(b2 - 0.4256508) < 1e-7
    r2 = b2 * r1 + (1 - b2) * (G2 ** 2).mean(axis=1)
    c2 = b2 * c1 + (1 - b2) * (G2 ** 2).mean(axis=0)
    v2 = np.outer(r2, c2) / r2.mean()
    u2 = G2 / np.sqrt(v2)
    u2 = u2 / max(1.0, math.sqrt(float(np.mean(u2 ** 2))))
    alpha2 = max(1e-3, math.sqrt(float(np.mean(th1 ** 2)))) * min(1e-2, 1.0 / math.sqrt(2.0))
    np.testing.assert_allclose(th2, th1 - alpha2 * u2.reshape(-1), rtol=1e-13)
    # each option alone changes the result, and the configured lr is not used under the relative step
    for kw in (dict(af_beta2_schedule=True), dict(af_clip=1.0), dict(af_relative_step=True)):
        ca = O.Config(1, 0, 1, 1, 32, lr=1e-3, beta2=0.9, **kw)
        cb = O.Config(1, 0, 1, 1, 32, lr=1e-3, beta2=0.9)
        sa, sb = O.step_init(ca, 4, 2, 2), O.step_init(cb, 4, 2, 2)
        ta, tb = th0, th0
        for G in (G1, G2):
            ta, tb = O.step(ta, G.reshape(-1), sa, ca, 2, 2), O.step(tb, G.reshape(-1), sb, cb, 2, 2)
        assert np.max(np.abs(ta - tb)) > 1e-6, kw
    # small update: no clipping happens (the factor is max(1, .))
    cs = O.Config(1, 0, 1, 1, 32, lr=1e-3, beta2=0.9, eps=10.0, af_clip=1.0)
    cn = O.Config(1, 0, 1, 1, 32, lr=1e-3, beta2=0.9, eps=10.0)
    np.testing.assert_array_equal(O.step(th0, G1.reshape(-1), O.step_init(cs, 4, 2, 2), cs, 2, 2),
                                  O.step(th0, G1.reshape(-1), O.step_init(cn, 4, 2, 2), cn, 2, 2))
    # relative step with a decoupled decay: the decay uses the same step size
    cw = O.Config(1, 0, 1, 1, 32, lr=7.0, beta2=0.9, eps=0.0, weight_decay=0.5, af_relative_step=True)
    sw = O.step_init(cw, 4, 2, 2)
    tw = O.step(th0, G1.reshape(-1), sw, cw, 2, 2)
    a = max(1e-3, math.sqrt(float(np.mean(th0 ** 2)))) * 1e-2
    vw = np.outer(0.1 * r1, 0.1 * c1) / (0.1 * 3.75)
    uw = G1 / np.sqrt(vw / (1 - 0.9))
    np.testing.assert_allclose(tw, th0 * (1 - a * 0.5) - a * uw.reshape(-1), rtol=1e-13)
