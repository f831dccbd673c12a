"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests retype the oracle's formulas in floating point: they use exact rational
arithmetic on the raw feature history (Eq. 2-3 as printed), closed forms, invariants, special
cases that reduce to a library routine (torch's bfloat16 conversion, Lagrange interpolation),
hand-computed examples and the one worked number the paper prints.
"""
import math
import os
from fractions import Fraction
from math import comb, factorial

import ctypes

import numpy as np
import pytest
import torch

from oracle import speca_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(x: torch.Tensor) -> np.ndarray:
    return x.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16).copy()


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def run_history(dtype, m, basis, times, feats):
    """Feed a raw feature history (oldest first) through the oracle; return planes and history."""
    n = feats[0].size
    planes = np.zeros((m + 1, n), dtype=O.np_dtype(dtype))
    hist = []
    for k, (t, f) in enumerate(zip(times, feats)):
        O.update_segment(dtype, m, basis, k, hist, t, np.ascontiguousarray(f), planes)
        hist = ([t] + hist)[: m + 1]
    return planes, hist


# ---------------------------------------------------------------------------------------------
# Eq. 2-3 as printed, in exact rationals, from the raw features on a uniform grid
# ---------------------------------------------------------------------------------------------

def eq3_delta(i, hist_at):
    """Delta^i F(x_t) = sum_j (-1)^(i-j) C(i,j) F(x_{t+jN}); hist_at(j) = F at t + j*N."""
    return sum(Fraction((-1) ** (i - j) * comb(i, j)) * hist_at(j) for j in range(i + 1))


def eq2_pred(m, N, k, hist_at):
    """F_pred(x_{t-k}) = F(x_t) + sum_{i=1..m} Delta^i F / (i! N^i) * (-k)^i."""
    s = Fraction(hist_at(0))
    for i in range(1, m + 1):
        s += eq3_delta(i, hist_at) * Fraction((-k) ** i, factorial(i) * N ** i)
    return s


@pytest.mark.parametrize("m", [1, 2, 3, 4])
@pytest.mark.parametrize("N", [1, 2, 4])
def test_taylor_basis_equals_printed_equations_in_rationals(m, N):
    rng = np.random.default_rng(100 * m + N)
    n = 37
    t = 40  # current step index; references at t + m*N, ..., t + N, t (time runs downwards)
    raw = {j: rng.integers(-50, 51, size=n) for j in range(m + 1)}  # F(x_{t+jN}), small integers
    times = [float(t + j * N) for j in range(m, -1, -1)]
    feats = [raw[j].astype(np.float32) for j in range(m, -1, -1)]
    planes, hist = run_history(O.F32, m, O.TAYLOR, times, feats)
    # stored planes are Delta^i / N^i (exact in binary for these N and integer features)
    for i in range(m + 1):
        for e in range(n):
            want = eq3_delta(i, lambda j: Fraction(int(raw[j][e]))) / Fraction(N ** i)
            assert Fraction(float(planes[i, e])) == want, (i, e)
    for k in [1, 2, 3, 5]:
        out = np.zeros(n, dtype=np.float32)
        O.forecast_segment(O.F32, m, O.TAYLOR, m + 1, hist, float(t - k), planes, out)
        for e in range(n):
            want = eq2_pred(m, N, k, lambda j: Fraction(int(raw[j][e])))
            got = float(out[e])
            assert abs(got - float(want)) <= 1.2e-7 * max(1.0, abs(float(want))), (k, e, got, float(want))


def test_counterexample_quadratic_is_not_reproduced_by_printed_equations():
    """f(s) = s^2, t = 0, N = 1, m = 2: Eq. 3 gives Delta^1 = 1, Delta^2 = 2 and Eq. 2 gives
    k^2 - k, not k^2. The oracle follows the printed equations."""
    m = 2
    times = [2.0, 1.0, 0.0]
    feats = [np.array([s * s], dtype=np.float32) for s in times]
    planes, hist = run_history(O.F32, m, O.TAYLOR, times, feats)
    assert planes[:, 0].tolist() == [0.0, 1.0, 2.0]
    for k in range(1, 6):
        out = np.zeros(1, dtype=np.float32)
        O.forecast_segment(O.F32, m, O.TAYLOR, 3, hist, float(-k), planes, out)
        assert out[0] == k * k - k


# ---------------------------------------------------------------------------------------------
# special cases of the forecast
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
def test_order_zero_is_plain_reuse_bit_for_bit(dtype):
    g = torch.Generator().manual_seed(1)
    x = torch.randn(4099, generator=g) * 7
    f = bf16_bits(x) if dtype == O.BF16 else x.numpy().copy()
    planes = np.zeros((1, f.size), dtype=f.dtype)
    O.update_segment(dtype, 0, O.TAYLOR, 0, [], 0.7, f, planes)
    assert np.array_equal(planes[0], f)
    out = np.zeros_like(f)
    O.forecast_segment(dtype, 0, O.TAYLOR, 1, [0.7], 0.3, planes, out)
    assert np.array_equal(out, f)
    # a later reference simply replaces the feature
    f2 = f[::-1].copy()
    O.update_segment(dtype, 0, O.TAYLOR, 1, [0.7], 0.6, f2, planes)
    O.forecast_segment(dtype, 0, O.TAYLOR, 2, [0.6], 0.1, planes, out)
    assert np.array_equal(out, f2)


@pytest.mark.parametrize("basis", [O.TAYLOR, O.NEWTON])
@pytest.mark.parametrize("m", [1, 2, 3])
def test_warm_up_uses_only_defined_orders(basis, m):
    """One reference -> reuse; two references -> straight line through them, whatever m is."""
    f0 = np.array([3.0, -8.0, 0.5], dtype=np.float32)
    f1 = np.array([5.0, -4.0, 0.25], dtype=np.float32)
    planes = np.full((m + 1, 3), 777.0, dtype=np.float32)  # garbage above the defined orders
    O.update_segment(O.F32, m, basis, 0, [], 8.0, f0, planes)
    out = np.zeros(3, dtype=np.float32)
    O.forecast_segment(O.F32, m, basis, 1, [8.0], 5.0, planes, out)
    assert np.array_equal(out, f0)
    O.update_segment(O.F32, m, basis, 1, [8.0], 6.0, f1, planes)
    O.forecast_segment(O.F32, m, basis, 2, [6.0, 8.0], 5.0, planes, out)
    assert out.tolist() == (f1 + (f1 - f0) / (6.0 - 8.0) * (5.0 - 6.0)).tolist()
    if m >= 2:
        assert np.all(planes[2] == 777.0)  # never written, never read


@pytest.mark.parametrize("basis", [O.TAYLOR, O.NEWTON])
@pytest.mark.parametrize("m", [1, 2, 3, 4])
def test_exact_for_degree_one_at_any_gaps(basis, m):
    rng = np.random.default_rng(5)
    a0 = rng.integers(-20, 21, size=11).astype(np.float64)
    a1 = rng.integers(-20, 21, size=11).astype(np.float64)
    times = [4.0, 3.5, 3.375, 2.0, 1.75, 1.0]  # dyadic, uneven
    feats = [(a0 + a1 * t).astype(np.float32) for t in times]
    planes, hist = run_history(O.F32, m, basis, times, feats)
    for tt in [0.5, 0.0, 1.0, 3.0, -2.25]:
        out = np.zeros(11, dtype=np.float32)
        O.forecast_segment(O.F32, m, basis, len(times), hist, tt, planes, out)
        assert np.array_equal(out.astype(np.float64), a0 + a1 * tt), tt


@pytest.mark.parametrize("m", [2, 3])
def test_taylor_basis_quadratic_residual_closed_form(m):
    """For f = a0 + a1 s + a2 s^2 and equal gaps g between the last references, backward
    difference quotients give D1 = f'(t) - a2 g, D2 = f''(t), so the printed forecast misses
    the truth by exactly -a2 * g * x (x = t_target - t_last)."""
    a0, a1, a2 = 3.0, -2.0, 5.0
    g = -0.25
    t_last = 2.0
    times = [t_last - j * g for j in range(m, -1, -1)]
    feats = [np.array([a0 + a1 * t + a2 * t * t], dtype=np.float32) for t in times]
    planes, hist = run_history(O.F32, m, O.TAYLOR, times, feats)
    for x in [-0.25, -0.5, -1.0, 0.125]:
        out = np.zeros(1, dtype=np.float32)
        O.forecast_segment(O.F32, m, O.TAYLOR, m + 1, hist, t_last + x, planes, out)
        tt = t_last + x
        truth = a0 + a1 * tt + a2 * tt * tt
        assert out[0] - truth == pytest.approx(-a2 * g * x, abs=1e-5)
    # the residual shrinks linearly with the reference gap
    res = []
    for gg in [-0.5, -0.25, -0.125]:
        ts = [t_last - j * gg for j in range(m, -1, -1)]
        fs = [np.array([a0 + a1 * t + a2 * t * t], dtype=np.float32) for t in ts]
        pl, hi = run_history(O.F32, m, O.TAYLOR, ts, fs)
        out = np.zeros(1, dtype=np.float32)
        O.forecast_segment(O.F32, m, O.TAYLOR, m + 1, hi, t_last - 0.5, pl, out)
        tt = t_last - 0.5
        res.append(float(out[0]) - (a0 + a1 * tt + a2 * tt * tt))
    assert res[0] == pytest.approx(2 * res[1], rel=1e-4) and res[1] == pytest.approx(2 * res[2], rel=1e-4)


@pytest.mark.parametrize("m", [1, 2, 3, 4])
def test_newton_basis_exact_for_degree_m_at_any_gaps(m):
    rng = np.random.default_rng(m)
    coef = rng.integers(-4, 5, size=(m + 1, 9)).astype(np.float64)
    times = [3.0, 2.5, 2.25, 1.5, 1.0, 0.875][: m + 2]

    def poly(t):
        return sum(coef[i] * t ** i for i in range(m + 1))

    feats = [poly(t).astype(np.float32) for t in times]
    planes, hist = run_history(O.F32, m, O.NEWTON, times, feats)
    for tt in [0.5, 0.25, 0.0, 2.0]:
        out = np.zeros(9, dtype=np.float32)
        O.forecast_segment(O.F32, m, O.NEWTON, len(times), hist, tt, planes, out)
        np.testing.assert_allclose(out.astype(np.float64), poly(tt), rtol=2e-6, atol=2e-5)


@pytest.mark.parametrize("m", [1, 2, 3])
def test_newton_basis_equals_lagrange_interpolation_in_rationals(m):
    """The Newton-form forecast is the unique polynomial of degree <= m through the last m+1
    references: compare with Lagrange's formula evaluated in exact rationals."""
    rng = np.random.default_rng(17 + m)
    times = [Fraction(8), Fraction(7), Fraction(11, 2), Fraction(5), Fraction(17, 4)][: m + 2]
    raw = [rng.integers(-30, 31, size=5) for _ in times]
    planes, hist = run_history(O.F32, m, O.NEWTON, [float(t) for t in times],
                               [r.astype(np.float32) for r in raw])
    nodes = times[-(m + 1):]
    vals = raw[-(m + 1):]
    for tt in [Fraction(4), Fraction(7, 2), Fraction(0)]:
        out = np.zeros(5, dtype=np.float32)
        O.forecast_segment(O.F32, m, O.NEWTON, len(times), hist, float(tt), planes, out)
        for e in range(5):
            want = Fraction(0)
            for a, ta in enumerate(nodes):
                w = Fraction(int(vals[a][e]))
                for c, tc in enumerate(nodes):
                    if c != a:
                        w *= (tt - tc) / (ta - tc)
                want += w
            assert float(out[e]) == pytest.approx(float(want), rel=1e-5, abs=1e-4)


def test_bases_coincide_up_to_order_one():
    rng = np.random.default_rng(3)
    times = [1.0, 0.9, 0.75]
    feats = [rng.standard_normal(64).astype(np.float32) for _ in times]
    pt, ht = run_history(O.F32, 1, O.TAYLOR, times, feats)
    pn, hn = run_history(O.F32, 1, O.NEWTON, times, feats)
    assert np.array_equal(pt, pn)
    a, b = np.zeros(64, np.float32), np.zeros(64, np.float32)
    O.forecast_segment(O.F32, 1, O.TAYLOR, 3, ht, 0.6, pt, a)
    O.forecast_segment(O.F32, 1, O.NEWTON, 3, hn, 0.6, pn, b)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("basis", [O.TAYLOR, O.NEWTON])
@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
def test_forecast_at_the_reference_time_returns_the_feature(basis, dtype):
    g = torch.Generator().manual_seed(9)
    m = 3
    times = [1.0, 0.8, 0.7, 0.65]
    feats = []
    for _ in times:
        x = torch.randn(257, generator=g)
        feats.append(bf16_bits(x) if dtype == O.BF16 else x.numpy().copy())
    planes, hist = run_history(dtype, m, basis, times, feats)
    out = np.zeros_like(feats[0])
    O.forecast_segment(dtype, m, basis, 4, hist, times[-1], planes, out)
    assert np.array_equal(out, feats[-1])


def test_zero_gap_is_refused_and_leaves_table_untouched():
    f = np.arange(8, dtype=np.float32)
    planes = np.zeros((3, 8), dtype=np.float32)
    O.update_segment(O.F32, 2, O.TAYLOR, 0, [], 1.0, f, planes)
    before = planes.copy()
    with pytest.raises(ZeroDivisionError):
        O.update_segment(O.F32, 2, O.TAYLOR, 1, [1.0], 1.0, f + 1, planes)
    assert np.array_equal(planes, before)
    with pytest.raises(RuntimeError):
        O.forecast_segment(O.F32, 2, O.TAYLOR, 0, [], 1.0, planes, np.zeros(8, np.float32))


# ---------------------------------------------------------------------------------------------
# storage rounding: bfloat16 round-to-nearest-even against torch's conversion
# ---------------------------------------------------------------------------------------------

def test_bf16_rounding_matches_library_conversion():
    g = torch.Generator().manual_seed(4)
    x = torch.cat([
        torch.randn(20000, generator=g) * torch.exp(torch.randn(20000, generator=g) * 8),
        torch.tensor([0.0, -0.0, 1.0, -1.0, 1.00390625, 1.01171875, 1.005859375, 3.3895314e38, -3.4e38,
                      1e-40, -1e-40, 9.1835e-41, 4.6e-41, 1.17549435e-38, float("inf"), float("-inf")]),
    ]).to(torch.float32)
    want = bf16_bits(x)
    got = np.array([O.to_bf16_bits(float(v)) for v in x.tolist()], dtype=np.uint16)
    assert np.array_equal(got, want)
    # exact ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert O.to_bf16_bits(1.0 + 2.0 ** -8) == 0x3F80
    assert O.to_bf16_bits(1.0 + 3 * 2.0 ** -8) == 0x3F82
    # a double just above the tie rounds up although its float32 rounding would be the tie itself
    assert O.to_bf16_bits(1.0 + 2.0 ** -8 + 2.0 ** -40) == 0x3F81
    assert O.to_bf16_bits(float("nan")) & 0x7FFF > 0x7F80


def test_stored_value_is_quantised_from_a_binary32_register():
    """fp32 accumulation, bf16 storage: c - d = 11 and gap = 0.98 - 1.0 (not exactly -0.02) give a
    quotient a hair below 550 in magnitude. 550 needs 9 significant bits, so it is an exact bfloat16
    tie between 548 and 552; held in a binary32 register it IS 550 and ties-to-even gives 552.
    Rounding the double directly would give 548."""
    f0 = np.array([O.to_bf16_bits(0.0)], dtype=np.uint16)
    f1 = np.array([O.to_bf16_bits(11.0)], dtype=np.uint16)
    planes, _ = run_history(O.BF16, 1, O.TAYLOR, [1.0, 0.98], [f0, f1])
    assert (0.98 - 1.0) != -0.02 and abs(11.0 / (0.98 - 1.0)) < 550.0
    assert float(bits_to_f64(planes[1])[0]) == -552.0
    # fp32 storage keeps the binary32 value itself
    pf, _ = run_history(O.F32, 1, O.TAYLOR, [1.0, 0.98], [np.zeros(1, np.float32), np.full(1, 11.0, np.float32)])
    assert float(pf[1, 0]) == float(np.float32(11.0 / (0.98 - 1.0))) == -550.0


def test_bf16_tables_round_once_per_stored_plane():
    """The difference chain runs on unrounded values: plane 2 is the rounding of the exact
    second quotient, not of a quotient of rounded first quotients."""
    vals = [1.0, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -6]  # bf16-exact features
    feats = [np.array([O.to_bf16_bits(v)], dtype=np.uint16) for v in vals]
    times = [3.0, 2.0, 1.0]
    planes, _ = run_history(O.BF16, 2, O.TAYLOR, times, feats)
    d1_old = Fraction(vals[1]) - Fraction(vals[0])
    d1_new = (Fraction(vals[2]) - Fraction(vals[1])) / Fraction(-1)
    # at the second update the old plane 1 was stored rounded; the new plane 1 is used unrounded
    d1_old_stored = Fraction(float(bits_to_f64(np.array([O.to_bf16_bits(float(d1_old / -1))], np.uint16))[0]))
    d2 = (d1_new - d1_old_stored) / Fraction(-1)
    assert int(planes[2, 0]) == O.to_bf16_bits(float(d2))
    assert int(planes[1, 0]) == O.to_bf16_bits(float(d1_new))
    assert int(planes[0, 0]) == O.to_bf16_bits(vals[2])


# ---------------------------------------------------------------------------------------------
# forecasts consumed as a sum (residual stream)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("basis", [O.TAYLOR, O.NEWTON, O.ADAMS_BASHFORTH])
@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
@pytest.mark.parametrize("m", [1, 2, 3, 4])   # every order: each has its own Adams-Bashforth coefficient
@pytest.mark.parametrize("layout", [O.LAYOUT_TABLES, O.LAYOUT_HISTORY])
def test_summed_forecast_of_one_entry_is_the_plain_forecast_bit_for_bit(basis, dtype, m, layout):
    g = torch.Generator().manual_seed(90 + basis)
    B, n = 2, 300
    cache = O.OracleCache([n, n], B, m, dtype, basis, layout=layout)
    for k, t in enumerate([1.0, 0.93, 0.9, 0.81, 0.79][: m + 1]):
        fs = [torch.randn(B, n, generator=g) for _ in range(2)]
        fs = [bf16_bits(f) if dtype == O.BF16 else f.numpy().copy() for f in fs]
        cache.update(fs, [t, t - 0.004])
        cache.commit_step()
    tt = [0.77, 0.75]
    for e in (0, 1):
        assert np.array_equal(cache.forecast_sum([e], tt), cache.forecast_entry(e, tt))


@pytest.mark.parametrize("layout", [O.LAYOUT_TABLES, O.LAYOUT_HISTORY])
def test_summed_forecast_is_the_sum_of_the_forecasts_in_exact_arithmetic(layout):
    # integer features, integer times, fp32 storage: every product and sum below is exact, so the sum
    # of the separately stored forecasts must equal the summed forecast, and adding a base adds it
    rng = np.random.default_rng(9)
    B, n, m, E = 2, 64, 2, 5
    cache = O.OracleCache([n] * E, B, m, O.F32, layout=layout)
    for t in (8.0, 6.0, 4.0):
        cache.update([rng.integers(-20, 20, (B, n)).astype(np.float32) * 8 for _ in range(E)], [t] * B)
        cache.commit_step()
    tt = [2.0, 0.0]
    parts = [as64(cache.forecast_entry(e, tt)) for e in range(E)]
    base = rng.integers(-100, 100, (B, n)).astype(np.float32)
    total = cache.forecast_sum(list(range(E)), tt)
    assert np.array_equal(as64(total), sum(parts))
    assert np.array_equal(as64(cache.forecast_sum([1, 3], tt, base=base)), parts[1] + parts[3] + base)
    # inactive samples keep what the output held
    out = np.full((B, n), 7.0, dtype=np.float32)
    cache.forecast_sum([0, 1], tt, active=[0, 1], out=out)
    assert np.all(out[0] == 7.0) and np.array_equal(as64(out[1]), (parts[0] + parts[1])[1])


def as64(a):
    return a.astype(np.float64)


# ---------------------------------------------------------------------------------------------
# the appendix's prediction-error bound, as a soft check (it equates differences with derivatives)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("m", [1, 2, 3])
def test_error_follows_the_taylor_remainder_and_the_appendix_bound(m):
    """Features c * exp(lambda * t): every derivative is lambda^i F, so the theorem's constant L is
    lambda. The forecast error must (i) stay below the theorem's leading term times (1 + L|x|) plus
    the O(h) finite-difference bias, (ii) approach the exact Taylor remainder
    |exp(lx) - sum (lx)^i / i!| linearly as the reference spacing h shrinks."""
    lam, x = 0.8, -0.5
    g = torch.Generator().manual_seed(3)
    c = (torch.rand(4000, generator=g) + 0.5).numpy().astype(np.float64)
    remainder = abs(math.exp(lam * x) - sum((lam * x) ** i / math.factorial(i) for i in range(m + 1)))
    gaps = []
    for h in (0.08, 0.04, 0.02):
        times = [1.0 - h * k for k in range(m + 1)]                     # oldest first, decreasing t
        feats = [(c * math.exp(lam * t)).astype(np.float32) for t in times]
        planes, hist = run_history(O.F32, m, O.TAYLOR, times, feats)
        out = np.zeros(c.size, np.float32)
        t0 = times[-1]
        O.forecast_segment(O.F32, m, O.TAYLOR, m + 1, hist, t0 + x, planes, out)
        truth = (c * math.exp(lam * (t0 + x))).astype(np.float32)
        now = (c * math.exp(lam * t0)).astype(np.float32)
        e_rel_to_now = float(np.linalg.norm(out.astype(np.float64) - truth) / np.linalg.norm(now))
        bound = (lam * abs(x)) ** (m + 1) / math.factorial(m + 1) * (1 + lam * abs(x)) + m * lam ** 2 * h * abs(x)
        assert e_rel_to_now <= bound, (m, h, e_rel_to_now, bound)
        gaps.append(abs(e_rel_to_now - remainder))
    # the distance to the exact Taylor remainder is the O(h) difference-quotient bias: it halves with h
    assert 1.5 < gaps[0] / gaps[1] < 2.6 and 1.5 < gaps[1] / gaps[2] < 2.6, gaps
    assert gaps[2] < 0.6 * m * lam ** 2 * 0.02 * abs(x) * 2


# ---------------------------------------------------------------------------------------------
# Adams-Bashforth draft model (appendix: named without a formula; pinned by the textbook method)
# ---------------------------------------------------------------------------------------------

AB_COEF = {1: [Fraction(1)], 2: [Fraction(3, 2), Fraction(-1, 2)],
           3: [Fraction(23, 12), Fraction(-16, 12), Fraction(5, 12)],
           4: [Fraction(55, 24), Fraction(-59, 24), Fraction(37, 24), Fraction(-9, 24)]}


@pytest.mark.parametrize("m", [1, 2, 3, 4])
@pytest.mark.parametrize("h", [-2, -1, 4])
def test_adams_bashforth_equals_textbook_formula_on_raw_history(m, h):
    """From the raw feature history on a uniform grid: slopes g_j = (F_j - F_{j+1}) / h, then the
    m-step Adams-Bashforth sum F_0 + x * sum b_j g_j, in exact rationals."""
    rng = np.random.default_rng(100 + m)
    n = 6
    times = [Fraction(16 + h * k) for k in range(m + 1)]            # oldest first: 16, 16+h, ...
    feats = [rng.integers(-40, 40, n).astype(np.float32) for _ in range(m + 1)]
    planes, hist = run_history(O.F32, m, O.ADAMS_BASHFORTH, [float(t) for t in times], feats)
    newest_first = feats[::-1]
    for x in (Fraction(h), Fraction(h, 2), Fraction(3 * h)):
        out = np.zeros(n, dtype=np.float32)
        O.forecast_segment(O.F32, m, O.ADAMS_BASHFORTH, m + 1, hist, float(times[-1] + x), planes, out)
        for e in range(n):
            g = [(Fraction(float(newest_first[j][e])) - Fraction(float(newest_first[j + 1][e]))) / h for j in range(m)]
            want = Fraction(float(newest_first[0][e])) + x * sum(b * gj for b, gj in zip(AB_COEF[m], g))
            assert float(out[e]) == pytest.approx(float(want), rel=1e-6, abs=1e-5)


def test_adams_bashforth_special_cases():
    rng = np.random.default_rng(7)
    n = 50
    times = [1.0, 0.9, 0.8, 0.7]
    feats = [rng.standard_normal(n).astype(np.float32) for _ in times]
    # one step: Euler with the latest slope = the Taylor basis at order 1, bit for bit
    pa, ha = run_history(O.F32, 1, O.ADAMS_BASHFORTH, times, feats)
    pt, ht = run_history(O.F32, 1, O.TAYLOR, times, feats)
    oa, ot = np.zeros(n, np.float32), np.zeros(n, np.float32)
    O.forecast_segment(O.F32, 1, O.ADAMS_BASHFORTH, 4, ha, 0.63, pa, oa)
    O.forecast_segment(O.F32, 1, O.TAYLOR, 4, ht, 0.63, pt, ot)
    assert np.array_equal(oa, ot)
    # the tables themselves are the Taylor-basis tables
    p3a, _ = run_history(O.F32, 3, O.ADAMS_BASHFORTH, times, feats)
    p3t, h3 = run_history(O.F32, 3, O.TAYLOR, times, feats)
    assert np.array_equal(p3a, p3t)
    # forecast at the reference time returns the feature; order 0 is plain reuse
    o = np.zeros(n, np.float32)
    O.forecast_segment(O.F32, 3, O.ADAMS_BASHFORTH, 4, h3, times[-1], p3a, o)
    assert np.array_equal(o, feats[-1])
    p0, h0 = run_history(O.F32, 0, O.ADAMS_BASHFORTH, times, feats)
    O.forecast_segment(O.F32, 0, O.ADAMS_BASHFORTH, 4, h0, 0.5, p0, o)
    assert np.array_equal(o, feats[-1])
    # a feature that is linear in t is extrapolated exactly at every step count
    lin = [(3.0 - 2.0 * t) * np.ones(n, dtype=np.float64) for t in times]
    for m in (1, 2, 3):
        pl, hl = run_history(O.F32, m, O.ADAMS_BASHFORTH, times, [v.astype(np.float32) for v in lin])
        O.forecast_segment(O.F32, m, O.ADAMS_BASHFORTH, 4, hl, 0.55, pl, o)
        assert np.allclose(o, 3.0 - 2.0 * 0.55, rtol=1e-5)


def test_adams_bashforth_on_a_quadratic_closed_form():
    """For F quadratic in t a secant slope is F' at the interval's midpoint, so the slopes are exact
    samples of the (linear) derivative at t_0 - h/2 and t_0 - 3h/2. The 2-step combination
    3/2 g_0 - 1/2 g_1 extrapolates a linear function half a step forward: it equals F'(t_0) exactly.
    Hence forecast = F(t_0) + x F'(t_0), and the distance to the truth is the closed form c x^2."""
    h = -0.125
    times = [1.0, 1.0 + h, 1.0 + 2 * h]
    a, bq, cq = 0.5, -1.25, 2.0
    F = lambda s: a + bq * s + cq * s * s
    dF = lambda s: bq + 2 * cq * s
    feats = [np.full(4, F(s), dtype=np.float32) for s in times]
    planes, hist = run_history(O.F32, 2, O.ADAMS_BASHFORTH, times, feats)
    out = np.zeros(4, np.float32)
    t0 = times[-1]
    for x in (h, 0.5 * h, 3 * h):
        O.forecast_segment(O.F32, 2, O.ADAMS_BASHFORTH, 3, hist, t0 + x, planes, out)
        assert np.allclose(out, F(t0) + x * dF(t0), rtol=1e-6)
        assert np.allclose(F(t0 + x) - out.astype(np.float64), cq * x * x, rtol=1e-4, atol=1e-7)


# ---------------------------------------------------------------------------------------------
# Eq. 4 and the accept rule
# ---------------------------------------------------------------------------------------------

def test_relative_error_hand_examples():
    f = np.array([5.0, 12.0], dtype=np.float32)       # norm 13
    p = f + np.array([3.0, 4.0], dtype=np.float32)    # difference norm 5
    assert O.rel_l2(O.F32, p, f) == pytest.approx(5.0 / (13.0 + 1e-8), rel=1e-15)
    assert O.rel_l2(O.F32, f, f) == 0.0
    z = np.zeros(2, dtype=np.float32)
    assert O.rel_l2(O.F32, z, f) == pytest.approx(13.0 / (13.0 + 1e-8), rel=1e-15)
    assert O.rel_l2(O.F32, p - f, z) == pytest.approx(5.0 / 1e-8, rel=1e-12)  # zero feature: only eps
    assert O.rel_l2(O.F32, z, z) == 0.0
    assert O.rel_l2(O.F32, p, f, eps=1.0) == pytest.approx(5.0 / 14.0, rel=1e-15)


def test_relative_error_properties():
    g = torch.Generator().manual_seed(11)
    f = torch.randn(5000, generator=g).numpy()
    p = (torch.randn(5000, generator=g) * 0.1).numpy() + f
    e = O.rel_l2(O.F32, p, f)
    assert O.rel_l2(O.F32, (4 * p).astype(np.float32), (4 * f).astype(np.float32)) == pytest.approx(e, rel=1e-7)
    delta = 2.0 ** -3
    fs = torch.from_numpy(f).to(torch.bfloat16).to(torch.float32).numpy()  # 8 significant bits
    pf = (fs * np.float32(1 + delta)).astype(np.float32)  # so that (1 + 2^-3) * f is exact in binary32
    nf = math.sqrt(math.fsum(float(v) ** 2 for v in fs))
    assert O.rel_l2(O.F32, pf, fs) == pytest.approx(delta * nf / (nf + 1e-8), rel=1e-12)
    # sensitive to which operand is the denominator
    assert O.rel_l2(O.F32, f, p) != pytest.approx(e, rel=1e-6)


@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
def test_relative_error_brute_force_in_rationals(dtype):
    g = torch.Generator().manual_seed(21)
    for n in [1, 2, 7, 16]:
        a, b = torch.randn(n, generator=g), torch.randn(n, generator=g)
        if dtype == O.BF16:
            p, f = bf16_bits(a), bf16_bits(b)
            pv, fv = bits_to_f64(p), bits_to_f64(f)
        else:
            p, f = a.numpy().copy(), b.numpy().copy()
            pv, fv = p.astype(np.float64), f.astype(np.float64)
        num = sum((Fraction(float(x)) - Fraction(float(y))) ** 2 for x, y in zip(pv, fv))
        den = sum(Fraction(float(y)) ** 2 for y in fv)
        want = math.sqrt(num) / (math.sqrt(den) + 1e-8)
        assert O.rel_l2(dtype, p, f) == pytest.approx(want, rel=1e-13)


# ---------------------------------------------------------------------------------------------
# the appendix's other error metrics (named there without formulas: pinned by the mathematics)
# ---------------------------------------------------------------------------------------------

OTHER_METRICS = [O.METRIC_L1, O.METRIC_LINF, O.METRIC_COSINE]


def test_other_metrics_hand_examples():
    f = np.array([3.0, -4.0, 1.0], dtype=np.float32)
    p = np.array([2.0, -6.0, 1.5], dtype=np.float32)      # differences -1, -2, 0.5
    assert O.rel_err(O.METRIC_L1, O.F32, p, f) == pytest.approx(3.5 / (8.0 + 1e-8), rel=1e-15)
    assert O.rel_err(O.METRIC_LINF, O.F32, p, f) == pytest.approx(2.0 / (4.0 + 1e-8), rel=1e-15)
    dot, pp, ff = 6.0 + 24.0 + 1.5, 4.0 + 36.0 + 2.25, 26.0
    assert O.rel_err(O.METRIC_COSINE, O.F32, p, f) == pytest.approx(
        1.0 - dot / (math.sqrt(pp) * math.sqrt(ff) + 1e-8), rel=1e-14)
    assert O.rel_err(O.METRIC_L2, O.F32, p, f) == O.rel_l2(O.F32, p, f)
    # two unit vectors in the plane at angle theta: cosine distance 1 - cos(theta)
    for theta in (0.0, 0.3, math.pi / 2, 2.5, math.pi):
        a = np.array([1.0, 0.0], dtype=np.float32)
        b = np.array([math.cos(theta), math.sin(theta)], dtype=np.float32)
        assert O.rel_err(O.METRIC_COSINE, O.F32, a, b) == pytest.approx(1.0 - math.cos(theta), abs=2e-7)
    # orthogonal -> 1, opposite -> 2
    assert O.rel_err(O.METRIC_COSINE, O.F32, np.array([1, 0], np.float32), np.array([0, 5], np.float32)) == pytest.approx(1.0, abs=1e-12)
    assert O.rel_err(O.METRIC_COSINE, O.F32, f, -f) == pytest.approx(2.0, abs=1e-7)


@pytest.mark.parametrize("metric", OTHER_METRICS)
def test_other_metrics_properties(metric):
    g = torch.Generator().manual_seed(31 + metric)
    f = torch.randn(4000, generator=g).to(torch.bfloat16).to(torch.float32).numpy()   # 8 significant bits
    p = (f + 0.1 * torch.randn(4000, generator=g).numpy()).astype(np.float32)
    e = O.rel_err(metric, O.F32, p, f)
    assert e > 0
    # forecast equal to the feature: zero error
    assert O.rel_err(metric, O.F32, f, f) == pytest.approx(0.0, abs=1e-7)
    # common scale factor (a power of two: exact) leaves the value unchanged
    assert O.rel_err(metric, O.F32, (4 * p).astype(np.float32), (4 * f).astype(np.float32)) == pytest.approx(e, rel=1e-7)
    delta = 2.0 ** -3
    pf = (f * np.float32(1 + delta)).astype(np.float32)   # exact in binary32
    if metric == O.METRIC_COSINE:
        assert O.rel_err(metric, O.F32, pf, f) == pytest.approx(0.0, abs=1e-7)      # same direction
        assert O.rel_err(metric, O.F32, f, p) == pytest.approx(e, rel=1e-9)         # symmetric
        assert O.rel_err(metric, O.F32, (3 * p).astype(np.float32), f) == pytest.approx(e, abs=1e-6)
    else:
        assert O.rel_err(metric, O.F32, pf, f) == pytest.approx(delta, rel=1e-7)    # p = (1+d) f -> |d|
        z = np.zeros_like(f)
        assert O.rel_err(metric, O.F32, z, f) == pytest.approx(1.0, rel=1e-7)       # p = 0 -> ||f||/(||f||+eps)
    # NaN anywhere -> NaN -> rejected
    q = p.copy()
    q[17] = np.nan
    assert math.isnan(O.rel_err(metric, O.F32, q, f))
    assert not O.accept(O.rel_err(metric, O.F32, q, f), 1e30)
    q = f.copy()
    q[5] = np.nan
    assert math.isnan(O.rel_err(metric, O.F32, p, q))


def test_norm_ordering_between_metrics():
    # for any vector ||x||_inf <= ||x||_2 <= ||x||_1 <= sqrt(n) ||x||_2 <= n ||x||_inf : checked on the
    # numerators by choosing the feature so that every denominator is 1 (a single unit entry)
    g = torch.Generator().manual_seed(5)
    n = 64
    f = np.zeros(n, dtype=np.float32)
    f[0] = 1.0
    d = torch.randn(n, generator=g).numpy().astype(np.float32)
    d[0] = 0.0
    p = (f + d).astype(np.float32)
    l1, l2, li = (O.rel_err(m, O.F32, p, f, eps=0.0) for m in (O.METRIC_L1, O.METRIC_L2, O.METRIC_LINF))
    assert li <= l2 <= l1 <= math.sqrt(n) * l2 <= n * li
    assert l1 == pytest.approx(float(np.abs(d.astype(np.float64)).sum()), rel=1e-12)
    assert li == pytest.approx(float(np.abs(d).max()), rel=1e-12)


@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
def test_other_metrics_brute_force_in_rationals(dtype):
    g = torch.Generator().manual_seed(41)
    for n in [1, 2, 7, 16]:
        a, b = torch.randn(n, generator=g), torch.randn(n, generator=g)
        if dtype == O.BF16:
            p, f = bf16_bits(a), bf16_bits(b)
            pv, fv = bits_to_f64(p), bits_to_f64(f)
        else:
            p, f = a.numpy().copy(), b.numpy().copy()
            pv, fv = p.astype(np.float64), f.astype(np.float64)
        P, F = [Fraction(float(x)) for x in pv], [Fraction(float(y)) for y in fv]
        l1 = float(sum(abs(x - y) for x, y in zip(P, F))) / (float(sum(abs(y) for y in F)) + 1e-8)
        li = float(max(abs(x - y) for x, y in zip(P, F))) / (float(max(abs(y) for y in F)) + 1e-8)
        cs = 1.0 - float(sum(x * y for x, y in zip(P, F))) / (
            math.sqrt(sum(x * x for x in P)) * math.sqrt(sum(y * y for y in F)) + 1e-8)
        assert O.rel_err(O.METRIC_L1, dtype, p, f) == pytest.approx(l1, rel=1e-13)
        assert O.rel_err(O.METRIC_LINF, dtype, p, f) == pytest.approx(li, rel=1e-13)
        assert O.rel_err(O.METRIC_COSINE, dtype, p, f) == pytest.approx(cs, abs=1e-13)


@pytest.mark.parametrize("metric", [O.METRIC_L2] + OTHER_METRICS)
def test_two_stage_metrics_agree_with_the_one_stage_ones_and_split_over_parts(metric):
    g = torch.Generator().manual_seed(77 + metric)
    f = torch.randn(3001, generator=g).numpy()
    p = (f + 0.05 * torch.randn(3001, generator=g).numpy()).astype(np.float32)
    whole = O.metric_sums(metric, O.F32, p, f)
    # the cosine distance is a difference of two numbers near 1: its absolute error is what the order
    # of summation (which depends on the thread count) moves
    tol = dict(rel=1e-12, abs=1e-13 if metric == O.METRIC_COSINE else 1e-15)
    assert O.metric_from_sums(metric, whole) == pytest.approx(O.rel_err(metric, O.F32, p, f), **tol)
    cut = 1234
    a = O.metric_sums(metric, O.F32, p[:cut].copy(), f[:cut].copy())
    b = O.metric_sums(metric, O.F32, p[cut:].copy(), f[cut:].copy())
    both = [max(x, y) for x, y in zip(a, b)] if metric == O.METRIC_LINF else [x + y for x, y in zip(a, b)]
    assert O.metric_from_sums(metric, both) == pytest.approx(O.rel_err(metric, O.F32, p, f), **tol)


@pytest.mark.parametrize("metric", [O.METRIC_L2] + OTHER_METRICS)
@pytest.mark.parametrize("where", ["forecast", "feature"])
def test_a_nan_element_makes_every_metric_nan_in_one_stage_and_in_two(metric, where):
    f = np.arange(1, 41, dtype=np.float32)
    p = f + 0.5
    (p if where == "forecast" else f)[17] = np.nan
    assert math.isnan(O.rel_err(metric, O.F32, p, f))
    assert math.isnan(O.metric_from_sums(metric, O.metric_sums(metric, O.F32, p, f)))
    # the part without the NaN is finite; combined with the other part the result is NaN again
    a, b = O.metric_sums(metric, O.F32, p[:10].copy(), f[:10].copy()), O.metric_sums(metric, O.F32, p[10:].copy(), f[10:].copy())
    assert all(math.isfinite(x) for x in a)
    both = [max(x, y) if not (math.isnan(x) or math.isnan(y)) else math.nan for x, y in zip(a, b)] \
        if metric == O.METRIC_LINF else [x + y for x, y in zip(a, b)]
    assert math.isnan(O.metric_from_sums(metric, both))
    assert not O.accept(math.nan, 1e30)


def test_accept_rule():
    assert O.accept(0.5, 0.5)            # equality accepts
    assert O.accept(0.0, 0.0)
    assert not O.accept(math.nextafter(0.5, 1.0), 0.5)
    assert O.accept(math.nextafter(0.5, 0.0), 0.5)
    assert not O.accept(float("nan"), 0.5)
    assert not O.accept(float("inf"), 1e30)
    f = np.array([1.0, float("nan")], dtype=np.float32)
    assert not O.accept(O.rel_l2(O.F32, f, f), 10.0)  # NaN anywhere rejects, even p == f


def test_threshold_schedule():
    assert O.tau_schedule(0.3, 0.5, 50, 50) == pytest.approx(0.3, rel=1e-15)       # t = T
    assert O.tau_schedule(0.3, 0.5, 0, 50) == pytest.approx(0.15, rel=1e-15)       # t = 0
    assert O.tau_schedule(0.1, 0.2, 25, 50) == pytest.approx(0.1 * math.sqrt(0.2), rel=1e-15)
    ts = [O.tau_schedule(0.1, 0.2, t, 50) for t in range(50, -1, -1)]
    assert all(a > b for a, b in zip(ts, ts[1:]))  # decays as t runs down
    assert ts[0] == pytest.approx(0.1) and ts[-1] == pytest.approx(0.02)


def test_speedup_matches_the_papers_worked_example():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "speedup_example.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 2
    for alpha, gamma, denom, s, nd in rows:
        alpha, gamma, denom, s, nd = float(alpha), float(gamma), float(denom), float(s), int(nd)
        got = O.speedup(alpha, gamma)
        assert 1.0 / got == pytest.approx(denom, rel=1e-12)
        assert round(got, nd) == pytest.approx(s)


def test_block_counts_match_printed_verification_ratios():
    from paper_2509_11628_b200 import workloads as W
    rows = [l.split() for l in open(os.path.join(GOLDEN, "gamma_blocks.txt")) if l.strip() and l[0] != "#"]
    for name, gamma, blocks in rows:
        gamma, blocks = float(gamma), int(blocks)
        assert 1.0 / blocks == pytest.approx(gamma, rel=0.03)
        w = W.BY_NAME[name]()
        if name == "dit_xl2":
            assert len(w.entries) == 2 * blocks
        else:
            duals = sum(1 for l in w.labels if l.endswith(".main"))
            singles = sum(1 for l in w.labels if l.startswith("S"))
            assert duals + singles == blocks


# ---------------------------------------------------------------------------------------------
# per-sample continuation
# ---------------------------------------------------------------------------------------------

def test_select_adaptive_hand_cases():
    # accept continues, reject stops, inactive stays inactive and is not counted
    act, cnt, idx = O.select_adaptive([1, 0, 1, 1], 5, 1, [0, 0, 2, 0], [1, 1, 1, 0])
    assert act == [1, 0, 1, 0] and cnt == [1, 0, 3, 0] and idx == [0, 2]
    # the forced activation period caps consecutive speculative steps
    act, cnt, idx = O.select_adaptive([1, 1], 3, 1, [1, 2], [1, 1])
    assert act == [1, 0] and cnt == [2, 3] and idx == [0]
    # a guidance pair shares its fate
    act, cnt, idx = O.select_adaptive([1, 0, 1, 1], 9, 2, [0, 0, 0, 0], [1, 1, 1, 1])
    assert act == [0, 0, 1, 1] and cnt == [1, 0, 1, 1] and idx == [2, 3]
    # sequential validation: once rejected, later accepts do not revive the sample
    act = [1]
    cnt = [0]
    trace = []
    for a in [1, 1, 0, 1, 1]:
        act, cnt, _ = O.select_adaptive([a], 99, 1, cnt, act)
        trace.append(act[0])
    assert trace == [1, 1, 0, 0, 0] and cnt == [2]


# ---------------------------------------------------------------------------------------------
# stateful wrapper: masks and per-sample histories
# ---------------------------------------------------------------------------------------------

def test_cache_masks_and_per_sample_history():
    rng = np.random.default_rng(8)
    B, m, n = 3, 2, 50
    c = O.OracleCache([n, n], B, m, O.F32)
    feats = lambda: [rng.standard_normal((B, n)).astype(np.float32) for _ in range(2)]
    f0 = feats()
    c.update(f0, [1.0, 1.0, 1.0]); c.commit_step()
    f1 = feats()
    c.update(f1, [0.9, 0.8, 0.9], mask=[1, 1, 0]); c.commit_step()
    assert c.n_refs == [2, 2, 1]
    assert c.t_hist[2] == [1.0] and c.t_hist[1] == [0.8, 1.0]
    # sample 2 was masked out: its table still holds the first feature only
    assert np.array_equal(c.planes[0][2, 0], f0[0][2])
    out = c.forecast_entry(1, [0.7, 0.7, 0.7])
    assert np.array_equal(out[2], f0[1][2])  # one reference: reuse
    want1 = f1[1][1] + (f1[1][1].astype(np.float64) - f0[1][1]) / (0.8 - 1.0) * (0.7 - 0.8)
    np.testing.assert_allclose(out[1], want1, rtol=1e-6, atol=1e-6)
    # inactive samples are left alone by forecast and verify
    sentinel = np.full((B, n), 42.0, dtype=np.float32)
    out2 = c.forecast_entry(0, [0.7] * 3, active=[0, 1, 0], out=sentinel.copy())
    assert np.all(out2[0] == 42.0) and np.all(out2[2] == 42.0) and not np.all(out2[1] == 42.0)
    err, acc, pred = c.verify(c.forecast_entry(1, [0.7] * 3), [0.7] * 3, [0.1] * 3, active=[1, 0, 1])
    assert err[0] == 0.0 and acc[0] == 1 and np.isnan(err[1]) and acc[1] == -1 and acc[2] == 1
    c.reset([0, 1, 0])
    assert c.n_refs == [2, 0, 1]


def test_cache_verify_scores_the_forecast_against_the_fresh_feature():
    # features linear in t with small-integer values: the forecast is exact in fp32 (degree 1), so a
    # fresh feature that is (1 + d) times the truth must score e = |d| / (1 + d), sample by sample
    B, m, n = 3, 2, 40
    rng = np.random.default_rng(15)
    a = rng.integers(-8, 9, (B, n)).astype(np.float64) * 4
    s = rng.integers(-8, 9, (B, n)).astype(np.float64) * 4
    s[:, 0] = 4.0                               # no sample is all zero
    feat = lambda t: (a + s * t).astype(np.float32)
    c = O.OracleCache([7, n], B, m, O.F32)      # verification entry = the last one
    for t in (8.0, 6.0, 4.0):
        c.update([np.zeros((B, 7), dtype=np.float32), feat(t)], [t] * B)
        c.commit_step()
    truth = feat(2.0)
    d = [0.0, 0.25, -0.5]
    fresh = np.stack([truth[b] * np.float32(1.0 + d[b]) for b in range(B)])
    err, acc, pred = c.verify(fresh, [2.0] * B, [0.3] * B)
    assert np.array_equal(pred, truth) and np.array_equal(pred, c.forecast_entry(1, [2.0] * B))
    for b in range(B):
        norm = math.sqrt(sum(float(x) ** 2 for x in truth[b]))           # ||truth||, exact integers
        assert err[b] == pytest.approx(abs(d[b]) * norm / ((1.0 + d[b]) * norm + 1e-8), rel=1e-12, abs=1e-15)
        assert err[b] == pytest.approx(abs(d[b]) / (1.0 + d[b]), rel=1e-9, abs=1e-15)   # epsilon is negligible here
    assert acc.tolist() == [1, 1, 0]            # 0 <= 0.3, 0.2 <= 0.3, 1.0 > 0.3
    # per-sample thresholds, and the l1 reading through the same call
    err1, acc1, _ = c.verify(fresh, [2.0] * B, [0.0, 0.1, 2.0], metric=O.METRIC_L1)
    assert err1 == pytest.approx(err, rel=1e-9, abs=1e-15) and acc1.tolist() == [1, 0, 1]   # up to epsilon's share


# ---------------------------------------------------------------------------------------------
# the cache that keeps raw features (history layout): Eq. 2-3 evaluated from them at forecast time
# ---------------------------------------------------------------------------------------------

def history_forecast(dtype, m, basis, times, feats, t_target):
    """times/feats oldest first; keeps the last m + 1 like the cache does."""
    hist_t = [float(t) for t in times][::-1][: m + 1]
    hist_f = [np.ascontiguousarray(f) for f in feats][::-1][: m + 1]
    out = np.zeros(hist_f[0].size, dtype=O.np_dtype(dtype))
    O.forecast_history_segment(dtype, m, basis, hist_t, float(t_target), hist_f, out)
    return out


@pytest.mark.parametrize("m", [1, 2, 3, 4])
@pytest.mark.parametrize("N", [1, 2, 3])
def test_history_layout_equals_printed_equations_in_rationals(m, N):
    # any N: nothing is stored between Eq. 3 and Eq. 2, so N = 3 (inexact quotients) works too
    rng = np.random.default_rng(500 + 10 * m + N)
    n, t = 23, 40
    raw = {j: rng.integers(-50, 51, size=n) for j in range(m + 1)}      # F(x_{t+jN})
    times = [float(t + j * N) for j in range(m, -1, -1)]
    feats = [raw[j].astype(np.float32) for j in range(m, -1, -1)]
    for k in [1, 2, 3, 5]:
        out = history_forecast(O.F32, m, O.TAYLOR, times, feats, t - k)
        for e in range(n):
            want = float(eq2_pred(m, N, k, lambda j: Fraction(int(raw[j][e]))))
            assert float(out[e]) == pytest.approx(want, rel=1.2e-7, abs=1.2e-7)


@pytest.mark.parametrize("m", [0, 1, 2, 3, 4])
def test_history_layout_equals_the_tables_when_nothing_rounds(m):
    # integer features and power-of-two gaps: every difference quotient is exact in binary32, so keeping
    # the quotients (tables) or the features (history) must give the same bits; more references than m + 1
    rng = np.random.default_rng(40 + m)
    a = O.OracleCache([16], 2, m, O.F32, O.TAYLOR)
    b = O.OracleCache([16], 2, m, O.F32, O.TAYLOR, layout=O.LAYOUT_HISTORY)
    t = 64.0
    for k in range(m + 4):
        f = [(rng.integers(-8, 8, (2, 16)) * 64).astype(np.float32)]
        t -= [1.0, 2.0, 4.0][k % 3]
        for c in (a, b):
            c.update(f, [t, t - 0.5])
            c.commit_step()
        tt = [t - 2.0, t - 1.0]
        assert np.array_equal(a.forecast_entry(0, tt), b.forecast_entry(0, tt)), k
        ea, aa, _ = a.verify(f[0], tt, [0.5, 0.5])
        eb, ab, _ = b.verify(f[0], tt, [0.5, 0.5])
        assert ea == pytest.approx(eb, rel=1e-12) and np.array_equal(aa, ab)   # same forecasts; the sum's order may vary


@pytest.mark.parametrize("basis", [O.TAYLOR, O.NEWTON, O.ADAMS_BASHFORTH])
@pytest.mark.parametrize("dtype", [O.F32, O.BF16])
def test_history_layout_tracks_the_tables_within_their_rounding(basis, dtype):
    # general inputs: the two layouts differ only by the tables' rounding of the stored quotients
    g = torch.Generator().manual_seed(60 + basis)
    m, B, n = 3, 2, 400
    a = O.OracleCache([n], B, m, dtype, basis)
    b = O.OracleCache([n], B, m, dtype, basis, layout=O.LAYOUT_HISTORY)
    for t in [1.0, 0.93, 0.9, 0.81, 0.78, 0.7]:
        f = torch.randn(B, n, generator=g)
        f = [bf16_bits(f) if dtype == O.BF16 else f.numpy().copy()]
        for c in (a, b):
            c.update(f, [t, t - 0.004])
            c.commit_step()
    x = a.forecast_entry(0, [0.66, 0.65])
    y = b.forecast_entry(0, [0.66, 0.65])
    xf, yf = (bits_to_f64(x), bits_to_f64(y)) if dtype == O.BF16 else (x.astype(np.float64), y.astype(np.float64))
    rel = np.linalg.norm(xf - yf) / np.linalg.norm(yf)
    assert 0 < rel < (3e-2 if dtype == O.BF16 else 1e-4)   # bf16 quotients amplified by (x / gap)^i


@pytest.mark.parametrize("m", [1, 2, 3, 4])
def test_history_layout_polynomial_exactness(m):
    rng = np.random.default_rng(70 + m)
    coef = rng.integers(-4, 5, size=(m + 1, 9)).astype(np.float64)
    times = [3.0, 2.5, 2.25, 1.5, 1.0, 0.875][: m + 2]
    poly = lambda t, deg: sum(coef[i] * t ** i for i in range(deg + 1))
    for tt in [0.5, 0.25, 0.0, 2.0]:
        # Newton reading: exact up to degree m at any gaps
        out = history_forecast(O.F32, m, O.NEWTON, times, [poly(t, m).astype(np.float32) for t in times], tt)
        np.testing.assert_allclose(out.astype(np.float64), poly(tt, m), rtol=2e-6, atol=2e-5)
        # Eq. 2-3 as printed: exact up to degree 1 at any gaps
        out = history_forecast(O.F32, m, O.TAYLOR, times, [poly(t, 1).astype(np.float32) for t in times], tt)
        np.testing.assert_allclose(out.astype(np.float64), poly(tt, 1), rtol=2e-6, atol=2e-5)
    # order 0 / one reference: plain reuse, bit for bit
    f = rng.standard_normal(9).astype(np.float32)
    assert np.array_equal(history_forecast(O.F32, m, O.TAYLOR, [1.0], [f], 0.3), f)
    assert np.array_equal(history_forecast(O.F32, 0, O.NEWTON, [1.0, 0.9], [f + 1, f], 0.3), f)


@pytest.mark.parametrize("m", [1, 2, 3, 4])
def test_history_layout_adams_bashforth_equals_textbook_formula(m):
    # uniform spacing h: F + x * sum_j b_j g_j with the slopes g_j = (F_j - F_{j+1}) / h taken from the raw features
    b = {1: [1.0], 2: [3 / 2, -1 / 2], 3: [23 / 12, -16 / 12, 5 / 12], 4: [55 / 24, -59 / 24, 37 / 24, -9 / 24]}[m]
    rng = np.random.default_rng(80 + m)
    h = -0.25
    times = [2.0 + h * k for k in range(m + 1)]                 # oldest first, time decreasing
    feats = [rng.integers(-20, 21, 11).astype(np.float32) for _ in times]
    x = -0.125
    out = history_forecast(O.F32, m, O.ADAMS_BASHFORTH, times, feats, times[-1] + x)
    newest_first = [f.astype(np.float64) for f in feats[::-1]]
    slopes = [(newest_first[j] - newest_first[j + 1]) / h for j in range(m)]
    want = newest_first[0] + x * sum(bj * gj for bj, gj in zip(b, slopes))
    np.testing.assert_allclose(out.astype(np.float64), want, rtol=1e-6, atol=1e-5)


def test_history_layout_cache_masks_resets_and_zero_gap():
    rng = np.random.default_rng(90)
    B, m, n = 3, 2, 12
    c = O.OracleCache([n], B, m, O.F32, O.TAYLOR, layout=O.LAYOUT_HISTORY)
    fs = [rng.integers(-9, 10, (B, n)).astype(np.float32) for _ in range(4)]
    c.update([fs[0]], [4.0] * B); c.commit_step()
    c.update([fs[1]], [3.0] * B, mask=[1, 0, 1]); c.commit_step()
    assert c.n_refs == [2, 1, 2] and len(c.hist[0][1]) == 1
    out = c.forecast_entry(0, [2.0] * B)
    assert np.array_equal(out[1], fs[0][1])                                   # one reference: reuse
    assert np.array_equal(out[0], 2 * fs[1][0] - fs[0][0])                     # two: linear extrapolation
    with pytest.raises(ZeroDivisionError):
        c.update([fs[2]], [3.0] * B)
    c.reset([1, 0, 0])
    c.update([fs[2]], [2.0] * B); c.commit_step()
    assert c.n_refs == [1, 2, 3] and len(c.hist[0][0]) == 1 and len(c.hist[0][2]) == 3
    out = c.forecast_entry(0, [1.0] * B, active=[1, 1, 0], out=np.full((B, n), 7.0, dtype=np.float32))
    assert np.array_equal(out[0], fs[2][0]) and np.all(out[2] == 7.0)
    assert np.array_equal(out[1], fs[2][1] + (fs[2][1] - fs[0][1]) / (2.0 - 4.0) * (1.0 - 2.0))   # its references: t = 4 and t = 2


def test_unrounded_history_forecast_rounds_to_the_stored_one():
    """forecast_history_unrounded is the value oracle_forecast_history_segment rounds: rounding it (double ->
    binary32 -> storage, as the oracle's store does) must give that function's output bit for bit, and for
    order 1 on two hand-picked features it is the straight line through them."""
    rng = np.random.default_rng(5)
    for dtype in (O.F32, O.BF16):
        for m in (1, 2, 3):
            t_hist = [0.7, 0.8, 0.95, 1.0][: m + 1]
            if dtype == O.F32:
                hist = [rng.standard_normal(257).astype(np.float32) for _ in range(m + 1)]
            else:
                hist = [(rng.standard_normal(257).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16) for _ in range(m + 1)]
            raw = O.forecast_history_unrounded(dtype, m, O.TAYLOR, t_hist, 0.64, hist)
            want = np.zeros(257, dtype=O.np_dtype(dtype))
            O.forecast_history_segment(dtype, m, O.TAYLOR, t_hist, 0.64, hist, want)
            got = np.zeros(257, dtype=O.np_dtype(dtype))
            O.lib().oracle_round_store(dtype, 257, raw.ctypes.data_as(ctypes.c_void_p), got.ctypes.data_as(ctypes.c_void_p))
            assert np.array_equal(got, want)
    a, b = np.array([3.0], dtype=np.float32), np.array([1.0], dtype=np.float32)   # f(0.5) = 3, f(1.0) = 1: slope -4
    raw = O.forecast_history_unrounded(O.F32, 1, O.TAYLOR, [0.5, 1.0], 0.25, [a, b])
    assert raw[0] == pytest.approx(4.0, abs=1e-12)
