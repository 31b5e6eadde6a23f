"""Population distortion of the Cubic level family (Section 3) -- oracle side, test infrastructure.

D_B(s, a, b) of Eq. explicit-cubic-risk evaluated with the closed-form cell moments of
Eq. reference-cell-moments for the three unit-variance reference sources, plus a Monte
Carlo estimate of the same quantity (Section 3.4).  Used only to pin the oracle's level
function and nearest-level rule against the paper's tables and closed forms.
"""
from __future__ import annotations

import math

import numpy as np

SQRT3 = math.sqrt(3.0)
BETA = 1.0 / math.sqrt(2.0)


def _phi(x):
    return math.exp(-0.5 * x * x) / math.sqrt(2.0 * math.pi) if math.isfinite(x) else 0.0


def _Phi(x):
    return 0.5 * (1.0 + math.erf(x / math.sqrt(2.0))) if math.isfinite(x) else 1.0


def cell_moments(dist: str, lo: float, hi: float):
    """(mu0, mu1, mu2) = integral over [lo, hi] of x^r f(x) dx on the positive half line
    (Eq. reference-cell-moments); hi may be +inf (upper-endpoint terms vanish)."""
    if dist == "uniform":
        lo_c, hi_c = min(max(lo, 0.0), SQRT3), min(max(hi, 0.0), SQRT3)
        return tuple((hi_c ** (r + 1) - lo_c ** (r + 1)) / (2.0 * SQRT3 * (r + 1)) for r in range(3))
    if dist == "gaussian":
        mu0 = _Phi(hi) - _Phi(lo)
        mu1 = _phi(lo) - _phi(hi)
        up = hi * _phi(hi) if math.isfinite(hi) else 0.0
        mu2 = mu0 + lo * _phi(lo) - up
        return mu0, mu1, mu2
    if dist == "laplace":
        El = math.exp(-lo / BETA)
        if math.isfinite(hi):
            Eu = math.exp(-hi / BETA)
            t0, t1, t2 = Eu, (hi + BETA) * Eu, (hi * hi + 2 * BETA * hi + 2 * BETA * BETA) * Eu
        else:
            t0 = t1 = t2 = 0.0
        mu0 = 0.5 * (El - t0)
        mu1 = 0.5 * ((lo + BETA) * El - t1)
        mu2 = 0.5 * ((lo * lo + 2 * BETA * lo + 2 * BETA * BETA) * El - t2)
        return mu0, mu1, mu2
    raise ValueError(dist)


def normalised_levels(B: int, a: float, b: float):
    """R_i(a,b) = r_i + a u_i + b v_i with r = t^3, u = t - t^3, v = t^2 - t^3 (Eq. cubic-basis,
    Eq. affine-cubic-level), i = 0..M."""
    M = (1 << (B - 1)) - 1
    out = []
    for i in range(M + 1):
        t = i / M
        out.append(t ** 3 + a * (t - t ** 3) + b * (t * t - t ** 3))
    return out


def population_distortion(dist: str, B: int, s: float, a: float, b: float) -> float:
    """D_B(s,a,b) = 2 sum_i [mu2 - 2 s R_i mu1 + s^2 R_i^2 mu0] over the cells (h_{i-1}, h_i),
    h_i = s (R_i + R_{i+1}) / 2, h_{-1} = 0, h_M = inf (Eq. explicit-cubic-risk)."""
    R = normalised_levels(B, a, b)
    M = len(R) - 1
    total = 0.0
    lo = 0.0
    for i in range(M + 1):
        hi = s * (R[i] + R[i + 1]) / 2.0 if i < M else math.inf
        mu0, mu1, mu2 = cell_moments(dist, lo, hi)
        total += mu2 - 2.0 * s * R[i] * mu1 + s * s * R[i] * R[i] * mu0
        lo = hi
    return 2.0 * total


def joint_population_distortion(dist: str, B: int, s: float, z, zt) -> float:
    """D_B^joint(s,a,b) of Eq. carrier-aware-population-objective for given normalised continuous
    levels z_i and carrier-grid levels zt_i (every code must own a cell: increasing boundaries):
    2 sum_i integral over (h_{i-1}, h_i) of [(x - s z_i)^2 + (x - s zt_i)^2] / 2 f(x) dx with the
    boundaries of Eq. carrier-aware-boundary, expanded in the cell moments of
    Eq. reference-cell-moments."""
    M = len(z) - 1
    h = [0.5 * s * ((z[i + 1] ** 2 + zt[i + 1] ** 2) - (z[i] ** 2 + zt[i] ** 2)) / ((z[i + 1] + zt[i + 1]) - (z[i] + zt[i]))
         for i in range(M)]
    assert all(h[i + 1] > h[i] for i in range(M - 1)), "a code owns no cell"
    total, lo = 0.0, 0.0
    for i in range(M + 1):
        hi = h[i] if i < M else math.inf
        mu0, mu1, mu2 = cell_moments(dist, lo, hi)
        for lev in (z[i], zt[i]):
            total += 0.5 * (mu2 - 2.0 * s * lev * mu1 + s * s * lev * lev * mu0)
        lo = hi
    return 2.0 * total


def best_scale(dist: str, B: int, a: float, b: float, lo: float = 0.05, hi: float = 20.0):
    """min over s of D_B(s, a, b): coarse scan then golden-section refinement."""
    grid = np.geomspace(lo, hi, 400)
    vals = [population_distortion(dist, B, float(s), a, b) for s in grid]
    i = int(np.argmin(vals))
    l, r = grid[max(i - 1, 0)], grid[min(i + 1, len(grid) - 1)]
    gr = (math.sqrt(5.0) - 1.0) / 2.0
    c, d = r - gr * (r - l), l + gr * (r - l)
    fc, fd = population_distortion(dist, B, c, a, b), population_distortion(dist, B, d, a, b)
    for _ in range(200):
        if fc < fd:
            r, d, fd = d, c, fc
            c = r - gr * (r - l)
            fc = population_distortion(dist, B, c, a, b)
        else:
            l, c, fc = c, d, fd
            d = l + gr * (r - l)
            fd = population_distortion(dist, B, d, a, b)
        if abs(r - l) < 1e-12:
            break
    s = 0.5 * (l + r)
    return s, population_distortion(dist, B, s, a, b)


def monte_carlo_distortion(samples: np.ndarray, levels_nonneg: np.ndarray):
    """Empirical mean squared error (and its standard error) of assigning each sample to its
    nearest signed level (Section 3.4).  ``levels_nonneg`` are the increasing non-negative
    levels; the codebook is their symmetric extension."""
    u = np.abs(samples)
    mids = 0.5 * (levels_nonneg[:-1] + levels_nonneg[1:])
    idx = np.searchsorted(mids, u, side="left")
    err2 = (u - levels_nonneg[idx]) ** 2
    return float(err2.mean()), float(err2.std(ddof=1) / math.sqrt(err2.size))
