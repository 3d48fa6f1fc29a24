"""The UOS quantization-error objective, evaluated numerically (test infrastructure only).

Section 4.1: E(x) = int_0^x (v - Pi(v))^2 dv, D(x) = E(x) / x^3 (Eq. 15),
J(q) = E[D(X_q)] = int_{q/2}^{q} D(x) g(x) dx (Eq. 17) with the wrapped density
g(x) = H(log2 x) / (x ln 2) (Eq. 18), and Delta(q) = E(q) - 8 E(q/2) (Eq. 29).

Nothing here is used by the quantizer; it exists so that the boundary 7.25 built into the
UOS rule can be recovered by brute force from the definition of the objective.
"""
from __future__ import annotations

import math
from fractions import Fraction

import numpy as np

GRID = (0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0)


def project(v):
    """Nearest point of the finite non-negative E2M1 grid (saturating at 6). Ties are measure zero."""
    v = np.asarray(v, dtype=np.float64)
    g = np.asarray(GRID)
    return g[np.abs(v[..., None] - g).argmin(axis=-1)]


def E_exact(x) -> Fraction:
    """E(x) by exact integration over the decision intervals (Appendix B, Eq. 41)."""
    x = Fraction(x)
    grid = [Fraction(g) for g in (0, Fraction(1, 2), 1, Fraction(3, 2), 2, 3, 4, 6)]
    cuts = [Fraction(0)] + [(a + b) / 2 for a, b in zip(grid[:-1], grid[1:])] + [None]
    total = Fraction(0)
    for r, a, b in zip(grid, cuts[:-1], cuts[1:]):
        hi = x if (b is None or x < b) else b
        if hi > a:
            total += ((hi - r) ** 3 - (a - r) ** 3) / 3
    return total


def E_numeric(x: float, n: int = 200001) -> float:
    """E(x) by composite Simpson on the raw integrand (no knowledge of the intervals)."""
    if x <= 0:
        return 0.0
    v = np.linspace(0.0, x, n)
    f = (v - project(v)) ** 2
    h = x / (n - 1)
    return float(h / 3 * (f[0] + f[-1] + 4 * f[1:-1:2].sum() + 2 * f[2:-1:2].sum()))


def E_float(x) -> np.ndarray:
    """E(x) in float64, vectorized: the same interval sum as E_exact (Appendix B, Eq. 41)."""
    x = np.asarray(x, dtype=np.float64)
    g = np.asarray(GRID)
    lo = np.concatenate([[0.0], (g[:-1] + g[1:]) / 2])
    hi = np.concatenate([(g[:-1] + g[1:]) / 2, [np.inf]])
    top = np.clip(x[..., None], lo, hi)                    # integrate each cell from lo to min(x, hi)
    return (((top - g) ** 3 - (lo - g) ** 3) / 3).sum(axis=-1)


def D(x):
    x = np.asarray(x, dtype=np.float64)
    return E_float(x) / x ** 3


def Delta(q) -> Fraction:
    q = Fraction(q)
    return E_exact(q) - 8 * E_exact(q / 2)


def J(q: float, H=None, n: int = 4001) -> float:
    """J(q) with t = log2 x:  int_{log2 q - 1}^{log2 q} D(2^t) H(t) dt  (H has period one, mean one)."""
    t1 = math.log2(q)
    t = np.linspace(t1 - 1.0, t1, n)
    w = np.ones_like(t) if H is None else np.asarray(H(t), dtype=np.float64)
    f = D(np.exp2(t)) * w
    h = 1.0 / (n - 1)
    return float(h / 3 * (f[0] + f[-1] + 4 * f[1:-1:2].sum() + 2 * f[2:-1:2].sum()))


def wrapped_gaussian_H(sigma: float, mu: float = 0.0, terms: int = 50):
    """Periodized density of U ~ N(mu, sigma^2) via its Fourier series (Appendix D, Eq. 52)."""
    def H(t):
        t = np.asarray(t, dtype=np.float64)
        return 1.0 + 2.0 * sum(math.exp(-2 * math.pi ** 2 * n * n * sigma * sigma)
                               * np.cos(2 * math.pi * n * (t - mu)) for n in range(1, terms))
    return H


def first_harmonic(sigma: float) -> float:
    """a_1(sigma) = 2 exp(-2 pi^2 sigma^2) (Appendix D, Eq. 53)."""
    return 2.0 * math.exp(-2.0 * math.pi ** 2 * sigma ** 2)
