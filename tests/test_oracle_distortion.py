"""Population distortion of the oracle's level family against the paper's closed forms, printed
tables and a Monte Carlo estimate (Section 3).  CPU only."""
import math

import numpy as np
import pytest

import datagen
import oracle
from oracle.distortion import best_scale, monte_carlo_distortion, population_distortion
from conftest import read_table


@pytest.mark.parametrize("B", range(2, 9))
def test_uniform_closed_form(B):
    # Eq. uniform-solution: s* = sqrt(3)(1 - 1/L), (a, b) = (1, 0), D* = 1/L^2, L = 2^B - 1.
    L = (1 << B) - 1
    s_star = math.sqrt(3.0) * (1.0 - 1.0 / L)
    D = population_distortion("uniform", B, s_star, 1.0, 0.0)
    assert abs(D - 1.0 / L ** 2) < 1e-14
    s_opt, D_opt = best_scale("uniform", B, 1.0, 0.0, 0.3, 3.0)
    assert abs(s_opt - s_star) < 1e-5 and abs(D_opt - D) < 1e-12
    printed = {int(r[0]): float(r[1]) for r in read_table("uniform_analytic.txt")}
    row = [r for r in read_table("uniform_analytic.txt") if int(r[0]) == B][0]
    assert abs(D - printed[B]) <= 0.51 * 10.0 ** (-len(row[1].split(".")[1]))  # half a unit of the last printed digit


def _digits_close(value, printed_str):
    """value agrees with a printed decimal to its last printed digit (half a unit, plus slack
    for the four-digit rounding of the printed a*, b*)."""
    printed = float(printed_str)
    frac = printed_str.split(".")[1]
    return abs(value - printed), 10.0 ** (-len(frac))


@pytest.mark.parametrize("row", read_table("population_tables.txt"), ids=lambda r: f"{r[0]}-B{r[1]}")
def test_population_tables(row):
    # Section 3.3 tables: D_C at the printed (a*, b*) with s optimised, and D_INT at (1, 0).
    dist, B, a, b = row[0], int(row[1]), float(row[2]), float(row[3])
    _, D_C = best_scale(dist, B, a, b)
    _, D_INT = best_scale(dist, B, 1.0, 0.0)
    err, unit = _digits_close(D_C, row[5])
    # printed (a*, b*) carry four decimals: the optimum is flat, allow 3 units of the last digit
    assert err <= 3 * unit, (D_C, row[5])
    err, unit = _digits_close(D_INT, row[6])
    assert err <= 1 * unit, (D_INT, row[6])
    D_LM = float(row[4])
    assert D_LM <= D_C * (1 + 1e-5) and D_C <= D_INT * (1 + 1e-9)  # Eq. cubic-sandwich


@pytest.mark.parametrize("dist", ["uniform", "gaussian", "laplace"])
@pytest.mark.parametrize("B", [2, 4, 8])
def test_monte_carlo_agrees(dist, B):
    # Section 3.4: nearest-level assignment of 2,000,000 samples against the cell-moment value.
    if dist == "uniform":
        a, b = 1.0, 0.0
    else:
        rows = {(r[0], int(r[1])): r for r in read_table("population_tables.txt")}
        a, b = float(rows[(dist, B)][2]), float(rows[(dist, B)][3])
    s, D = best_scale(dist, B, a, b)
    g = datagen.stream(1234, f"mc-{dist}-{B}")
    n = 2_000_000
    if dist == "uniform":
        x = datagen.uniform_pm(g, n, math.sqrt(3.0))
    elif dist == "gaussian":
        x = datagen.normal(g, n)
    else:
        x = datagen.laplace(g, n, 1.0 / math.sqrt(2.0))
    # levels from the oracle's own level function (binary16 a, b would perturb: use s only through fp64 path)
    from oracle.distortion import normalised_levels
    lev = s * np.array(normalised_levels(B, a, b))
    D_mc, se = monte_carlo_distortion(x, lev)
    assert abs(D - D_mc) <= 4.0 * se, (D, D_mc, se)


def test_distortion_uses_oracle_levels_consistently():
    # the fp64 curve in distortion.py and cqo_levels agree for binary16-representable (a, b)
    from oracle.distortion import normalised_levels
    for B in (3, 4, 8):
        a, b = np.float16(0.75), np.float16(-0.375)
        lev = oracle.levels(B, np.float32(1.0), a, b)
        R = normalised_levels(B, float(a), float(b))
        assert np.allclose(lev, R, rtol=0, atol=1e-15)
