"""Pins for oracle/uos_theory.py and, through it, for the 7.25 boundary the quantizer uses.  CPU only."""
import math
import os
from fractions import Fraction as F

import numpy as np

from oracle import mxfp4, uos_theory as th

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rows(name):
    for line in open(os.path.join(GOLD, name)):
        if line.startswith("#") or not line.strip():
            continue
        yield line.split()


def test_cumulative_error_table():
    # Appendix B table: exact interval integration and blind numeric quadrature both give the printed values
    for x, frac in rows("e2m1_cumulative_error.txt"):
        want = F(frac)
        assert th.E_exact(F(x)) == want
        assert abs(th.E_numeric(float(x)) - float(want)) < 2e-9


def test_error_above_six_closed_form():
    # Eq. 42: E(q) = 7/8 + (q - 6)^3 / 3 for q >= 6
    for q in (F(6), F(13, 2), F(7), F(29, 4), F(8), F(12)):
        assert th.E_exact(q) == F(7, 8) + (q - 6) ** 3 / 3
    assert abs(th.E_numeric(7.25) - (7 / 8 + 1.25 ** 3 / 3)) < 1e-8


def test_delta_matches_all_nine_rows_and_signs():
    for lo, hi, expr, sign in rows("delta_piecewise.txt"):
        lo = F(lo)
        hi = F(1000) if hi == "inf" else F(hi)
        for k in range(1, 12):
            q = lo + (hi - lo) * F(k, 12)
            want = eval(expr, {"q": q, "F": F})
            got = th.Delta(q)
            assert got == want, (lo, hi, q, got, want)
            if sign == "-":
                assert got < 0
            elif sign == "+":
                assert got > 0
            elif sign == "0":
                assert got == 0
        assert th.Delta(hi) == eval(expr, {"q": hi, "F": F})          # right end is closed


def test_delta_on_6_8_and_root():
    # Eq. 30
    for q in (F(6), F(13, 2), F(7)):
        assert th.Delta(q) == F(-1, 8)
    for q in (F(7), F(36, 5), F(29, 4), F(15, 2), F(8)):
        assert th.Delta(q) == (4 * q - 29) * (4 * q - 27) / 8
    assert th.Delta(F(29, 4)) == 0
    assert th.Delta(F(29, 4) - F(1, 1000)) < 0 < th.Delta(F(29, 4) + F(1, 1000))
    assert 864 ** 2 - 4 * 48 * 3983 == -18240                          # Appendix C discriminant


def test_brute_force_scan_of_objective_recovers_7_25():
    # Theorem 1: argmin_q J(q) = 29/4 for any wrapped density; scan q in [5, 9] step 0.01
    qs = np.round(np.arange(5.0, 9.0001, 0.01), 2)
    densities = {
        "log-uniform": None,
        "wrapped gaussian 0.2": th.wrapped_gaussian_H(0.2, 0.3),
        "wrapped gaussian 0.3": th.wrapped_gaussian_H(0.3, 0.77),
        "cosine": lambda t: 1.0 + 0.8 * np.cos(2 * math.pi * (np.asarray(t) - 0.1)),
    }
    for name, H in densities.items():
        j = np.array([th.J(float(q), H, n=2001) for q in qs])
        assert qs[j.argmin()] == 7.25, (name, qs[j.argmin()])
        # monotone on both sides within numerical noise (Appendix C)
        i = j.argmin()
        assert np.all(np.diff(j[:i + 1]) < 1e-12) and np.all(np.diff(j[i:]) > -1e-12)


def test_boundary_used_by_the_quantizer_is_the_scanned_optimum():
    assert mxfp4.UOS.q == 7.25 and mxfp4.UOS.family == "ceil"
    assert mxfp4.OCP.q == 8.0 and mxfp4.OCP.family == "floor"


def test_first_harmonic_table():
    for sigma, a1 in rows("first_harmonic.txt"):
        got = th.first_harmonic(float(sigma))
        assert abs(got - float(a1)) <= 0.6 * 10 ** (math.floor(math.log10(float(a1))) - (2 if float(a1) < 1e-6 else 3)) \
            or abs(got - float(a1)) < 6e-5
    # and the series used for the scan has that first coefficient
    H = th.wrapped_gaussian_H(0.3, 0.0)
    t = np.linspace(0, 1, 2000, endpoint=False)
    c1 = 2 * np.mean(H(t) * np.cos(2 * math.pi * t))
    assert abs(c1 - th.first_harmonic(0.3)) < 1e-9


def test_float_error_integral_equals_exact_one():
    xs = [F(k, 37) for k in range(0, 400)]
    got = th.E_float(np.array([float(x) for x in xs]))
    want = np.array([float(th.E_exact(x)) for x in xs])
    assert np.allclose(got, want, rtol=0, atol=1e-13)
