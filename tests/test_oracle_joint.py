"""Pins and invariants of the oracle's carrier-aware (dual-path) fitting, Section 4.3.  CPU only.

Each pin computes the quantity another way than the oracle does: an enumeration of every code
vector, the decision boundaries of Eq. carrier-aware-boundary, the stationarity of the joint loss in
s, the W1 / W2 and integer-grid special cases where the carrier projection is the identity."""
import itertools

import numpy as np
import pytest

import datagen
import oracle

ONE, ZERO = np.float16(1.0), np.float16(0.0)
SHAPES = [(0.6, -0.3), (0.45, 0.1), (1.0, 0.0), (0.8, -0.55)]


def joint_cost(w, k, B, s, a, b):
    lc, la = oracle.group_losses(w, B, s, a, b, k)
    return lc + la


@pytest.mark.parametrize("B", [3, 4, 6])
def test_carrier_grid_levels_are_the_rounded_continuous_levels(B):
    # Eq. carrier-grid: ztilde = round(127 z) / 127, and the carriers are what the A8 path multiplies by
    for a, b in SHAPES:
        z, zt = oracle.joint_levels(B, np.float16(a), np.float16(b))
        r = oracle.carriers(B, np.float16(a), np.float16(b)).astype(np.float64)
        assert np.array_equal(zt * 127.0, r)
        frac = 127.0 * z - np.floor(127.0 * z)
        clear = np.abs(frac - 0.5) > 1e-4            # away from rounding ties the fp32 sequence cannot differ
        assert np.array_equal(np.rint(127.0 * z)[clear], r[clear])
        assert np.all(np.abs(z - zt) <= 0.5 / 127 + 1e-6)


@pytest.mark.parametrize("B", [2, 3])
def test_joint_assignment_is_the_minimiser_by_enumeration(B):
    # every code vector of a tiny group is scored with the two reconstructions of
    # Eq. continuous-and-carrier-reconstruction; the assignment must reach the minimum
    M = (1 << (B - 1)) - 1
    rng = np.random.default_rng(5)
    G = 6 if B == 2 else 4
    for trial in range(6):
        w = rng.normal(0, 0.05, G).astype(np.float32)
        a, b = (ONE, ZERO) if B == 2 else (np.float16(0.55), np.float16(-0.2))
        s = np.float32(np.abs(w).max() * (0.7 + 0.05 * trial))
        k = oracle.assign_group_joint(w, B, s, a, b)
        best = min(joint_cost(w, np.array(kv, dtype=np.int8), B, s, a, b)
                   for kv in itertools.product(range(-M, M + 1), repeat=G))
        assert joint_cost(w, k, B, s, a, b) <= best * (1 + 1e-12) + 1e-30
        assert np.all(np.abs(k) <= M)


@pytest.mark.parametrize("B", [3, 4, 5])
def test_joint_assignment_follows_the_joint_boundaries(B):
    # Eq. carrier-aware-boundary: between adjacent codes the decision point is
    # h_i = (s/2) [(z_{i+1}^2 + zt_{i+1}^2) - (z_i^2 + zt_i^2)] / [(z_{i+1} + zt_{i+1}) - (z_i + zt_i)].
    # Where every code owns an interval (boundaries increasing), a weight strictly inside (h_{i-1}, h_i) gets code i.
    M = (1 << (B - 1)) - 1
    for a, b in SHAPES:
        a16, b16 = np.float16(a), np.float16(b)
        z, zt = oracle.joint_levels(B, a16, b16)
        s = np.float32(0.037)
        num = (z[1:] ** 2 + zt[1:] ** 2) - (z[:-1] ** 2 + zt[:-1] ** 2)
        den = (z[1:] + zt[1:]) - (z[:-1] + zt[:-1])
        h = 0.5 * float(s) * num / den
        if not np.all(np.diff(h) > 0):
            continue
        edges = np.concatenate([[0.0], h, [2.0 * float(s)]])
        mids = 0.5 * (edges[:-1] + edges[1:])
        w = np.concatenate([mids, -mids]).astype(np.float32)
        safe = np.minimum(mids - edges[:-1], edges[1:] - mids) > 1e-6
        k = oracle.assign_group_joint(w, B, s, a16, b16)
        want = np.concatenate([np.arange(M + 1), -np.arange(M + 1)])
        keep = np.concatenate([safe, safe])
        assert np.array_equal(k[keep], want[keep].astype(np.int8))
        # and these boundaries are not the continuous midpoints unless the carrier projection is exact
        mid_c = 0.5 * float(s) * (z[1:] + z[:-1])
        if np.any(np.abs(z - zt) > 1e-9):
            assert np.any(np.abs(h - mid_c) > 1e-12)


@pytest.mark.parametrize("B", [3, 4, 8])
def test_joint_scale_is_the_stationary_point_of_the_joint_loss(B):
    # Eq. carrier-aware-scale against the loss itself: L(s*) <= L(s* (1 +- eps)) and the central
    # difference of L at s* vanishes
    W = datagen.weights("laplace", 4, 128, seed=21, b=0.015)
    a16, b16 = np.float16(0.6), np.float16(-0.25)
    for row in W:
        w = row.astype(np.float32)
        k = oracle.assign_group_joint(w, B, np.float32(np.abs(w).max() * 0.8), a16, b16)
        s_star = oracle.joint_scale(w, k, B, a16, b16)
        z, zt = oracle.joint_levels(B, a16, b16)
        i = np.abs(k.astype(np.int64))
        u = np.abs(w.astype(np.float64))

        def loss(s):
            return float(np.sum((u - s * z[i]) ** 2 + (u - s * zt[i]) ** 2))
        assert loss(s_star) <= loss(s_star * (1 + 1e-4)) and loss(s_star) <= loss(s_star * (1 - 1e-4))
        eps = 1e-6 * s_star
        slope = (loss(s_star + eps) - loss(s_star - eps)) / (2 * eps)
        curv = 2.0 * float(np.sum(z[i] ** 2 + zt[i] ** 2))
        assert abs(slope) <= 1e-6 * curv * s_star
        # the stored (fp32) losses agree with the same sums
        lc, la = oracle.group_losses(w, B, np.float32(s_star), a16, b16, k)
        s32 = float(np.float32(s_star))
        assert lc + la == pytest.approx(loss(s32), rel=1e-12)


@pytest.mark.parametrize("B", [1, 2])
def test_w1_w2_levels_lie_on_the_carrier_grid(B):
    # Section 4.3: for W1 and W2 L_C = L_A8, the correction has no effect: the joint encoder returns
    # exactly what the continuous encoder returns
    W = datagen.weights("normal", 6, 256, seed=31, sigma=0.02)
    for effort in ("int_clipped", "fast"):
        kc, sc, ac, bc = oracle.encode(W, B, 64, effort)
        kj, sj, aj, bj = oracle.encode(W, B, 64, effort, objective="joint")
        assert np.array_equal(kc, kj) and np.array_equal(sc, sj)
        assert np.array_equal(ac.view(np.uint16), aj.view(np.uint16)) and np.array_equal(bc.view(np.uint16), bj.view(np.uint16))
    w = W[0, :64]
    lc, la = oracle.group_losses(w, B, sc[0, 0], ac[0, 0], bc[0, 0], kc[0, :64])
    assert lc == la


def test_integer_grid_at_w8_makes_both_assignments_agree():
    # B = 8, (a, b) = (1, 0): q(i/127) = i/127, so 127 q is an integer, ztilde = z, and the joint
    # assignment is the plain nearest-level assignment
    z, zt = oracle.joint_levels(8, ONE, ZERO)
    assert np.array_equal(z, zt)
    w = datagen.weights("normal", 1, 256, seed=41, sigma=0.02)[0]
    s = np.float32(np.abs(w).max())
    assert np.array_equal(oracle.assign_group(w, 8, s, ONE, ZERO), oracle.assign_group_joint(w, 8, s, ONE, ZERO))


@pytest.mark.parametrize("B", [3, 4, 5])
def test_joint_encoder_invariants(B):
    # (1) never worse, jointly, than the continuous encoder's answer; (2) no reserved pattern; (3) stored
    # curves strictly monotone; (4) its A8 error is not larger than the continuous answer's by more than
    # the continuous error it gives up: L_joint(joint) <= L_joint(cont)
    G = 64
    W = datagen.weights("laplace", 12, 256, seed=51, b=0.015)
    kc, sc, ac, bc = oracle.encode(W, B, G, "fast")
    kj, sj, aj, bj = oracle.encode(W, B, G, "fast", objective="joint")
    M = (1 << (B - 1)) - 1
    assert np.abs(kj).max() <= M
    tot_c = tot_j = a8_c = a8_j = 0.0
    for n in range(W.shape[0]):
        for g in range(W.shape[1] // G):
            w = W[n, g * G:(g + 1) * G]
            lc_c, la_c = oracle.group_losses(w, B, sc[n, g], ac[n, g], bc[n, g], kc[n, g * G:(g + 1) * G])
            lc_j, la_j = oracle.group_losses(w, B, sj[n, g], aj[n, g], bj[n, g], kj[n, g * G:(g + 1) * G])
            assert lc_j + la_j <= (lc_c + la_c) * (1 + 1e-9) + 1e-30
            assert oracle.shape_margin(float(aj[n, g]), float(bj[n, g])) > 0
            tot_c += lc_c + la_c; tot_j += lc_j + la_j; a8_c += la_c; a8_j += la_j
    assert tot_j <= tot_c
    # reporting quantity of Eq. carrier-aware-nrmse is well defined and below the INT8-grid-free bound 1
    nrmse = np.sqrt(tot_j / (2.0 * float(np.sum(W.astype(np.float64) ** 2))))
    assert 0 < nrmse < 1


@pytest.mark.parametrize("dist", ["gaussian", "laplace", "uniform"])
@pytest.mark.parametrize("B", [3, 4])
def test_joint_population_distortion_against_monte_carlo(dist, B):
    # Eq. carrier-aware-population-objective from closed-form cell moments and the joint boundaries, against
    # the empirical (L_C + L_A8) / (2 n) of the oracle's joint assignment on unit-variance samples
    from oracle import distortion
    a16, b16 = np.float16(0.6), np.float16(-0.25)
    z, zt = oracle.joint_levels(B, a16, b16)
    s = {3: 2.2, 4: 2.9}[B] if dist != "uniform" else 1.7
    want = distortion.joint_population_distortion(dist, B, s, list(z), list(zt))
    g = datagen.stream(77, f"mc-{dist}-{B}")
    n = 400_000
    x = {"gaussian": datagen.normal, "laplace": lambda gg, m: datagen.laplace(gg, m, 1.0 / np.sqrt(2.0)),
         "uniform": lambda gg, m: datagen.uniform_pm(gg, m, np.sqrt(3.0))}[dist](g, n).astype(np.float32)
    assert abs(float(np.var(x.astype(np.float64))) - 1.0) < 0.02          # the reference sources have unit variance
    k = oracle.assign_group_joint(x, B, np.float32(s), a16, b16)
    lc, la = oracle.group_losses(x, B, np.float32(s), a16, b16, k)
    got = (lc + la) / (2.0 * n)
    i = np.abs(k.astype(np.int64))
    per = 0.5 * ((np.abs(x.astype(np.float64)) - s * z[i]) ** 2 + (np.abs(x.astype(np.float64)) - s * zt[i]) ** 2)
    se = float(per.std(ddof=1) / np.sqrt(n))
    assert abs(got - want) <= 5.0 * se + 1e-6, (got, want, se)
    # and it differs from the continuous distortion at the same parameters whenever the projection moves a level
    cont = distortion.population_distortion(dist, B, s, float(a16), float(b16))
    assert want >= cont - 1e-12
