"""Pins and invariants of the oracle encoder (Section 4.1) and of the Dynamic-A8 reference
(Sections 4.3, 5.4).  CPU only."""
import itertools
import math

import numpy as np
import pytest

import datagen
import oracle
from conftest import read_table

ONE, ZERO = np.float16(1.0), np.float16(0.0)


@pytest.mark.parametrize("B", [2, 3, 4, 8])
def test_int_point_is_textbook_absmax_int(B):
    # restricted to (a, b) = (1, 0) with s = max|w|, the encoder is symmetric absmax INT:
    # k = round(w M / max|w|)
    M = (1 << (B - 1)) - 1
    W = datagen.weights("normal", 8, 256, seed=11, sigma=0.02)
    k, s, a, b = oracle.encode(W, B, 64, "int_absmax")
    assert np.all(a == ONE) and np.all(b == ZERO)
    Wg = W.reshape(8, 4, 64).astype(np.float64)
    amax = np.abs(Wg).max(axis=2)
    assert np.array_equal(s, amax.astype(np.float32))
    ref = Wg * M / amax[:, :, None]
    kref = np.sign(ref) * np.floor(np.abs(ref) + 0.5)
    ties = np.abs(np.abs(ref) - np.floor(np.abs(ref)) - 0.5) < 1e-9
    assert np.array_equal(k.reshape(8, 4, 64)[~ties], kref[~ties].astype(np.int8))


@pytest.mark.parametrize("B", [2, 3])
def test_nearest_level_assignment_is_sse_minimiser_brute_force(B):
    # for fixed (s, a, b) every code vector is enumerated on a tiny group
    M = (1 << (B - 1)) - 1
    rng = np.random.default_rng(3)
    G = 5 if B == 3 else 6
    for trial in range(6):
        w = rng.normal(0, 0.05, G).astype(np.float32)
        s, a, b = np.float32(0.09), np.float16(0.7 if B == 3 else 1.0), np.float16(-0.2 if B == 3 else 0.0)
        k = oracle.assign_group(w, B, s, a, b)
        best = min(oracle.group_sse(w, B, s, a, b, np.array(kv, np.int8))
                   for kv in itertools.product(range(-M, M + 1), repeat=G))
        assert abs(oracle.group_sse(w, B, s, a, b, k) - best) < 1e-15
        assert np.all(np.abs(k) <= M)


def test_least_squares_scale_is_optimal_for_fixed_codes():
    # after encoding, perturbing the stored scale cannot reduce the error by more than fp32 rounding allows
    W = datagen.weights("laplace", 4, 128, seed=5, b=0.015)
    for B in (3, 4, 6):
        k, s, a, b = oracle.encode(W, B, 128, "fast")
        for n in range(4):
            base = oracle.group_sse(W[n], B, s[n, 0], a[n, 0], b[n, 0], k[n])
            for f in (0.97, 0.99, 1.01, 1.03):
                assert oracle.group_sse(W[n], B, np.float32(s[n, 0] * f), a[n, 0], b[n, 0], k[n]) >= base * (1 - 1e-6)


def test_w1_scale_is_mean_abs_and_brute_force():
    W = datagen.weights("normal", 2, 64, seed=6, sigma=0.02)
    k, s, a, b = oracle.encode(W, 1, 32, "fast")
    assert set(np.unique(k)) <= {-1, 1}
    assert np.allclose(s, np.abs(W).reshape(2, 2, 32).mean(axis=2), rtol=1e-6)
    # brute force over a scale grid for one group
    w = W[0, :32].astype(np.float64)
    grid = np.linspace(0, 0.06, 6001)
    sse = [(np.abs(w) - g) @ (np.abs(w) - g) for g in grid]
    assert abs(grid[int(np.argmin(sse))] - s[0, 0]) < 2e-5


@pytest.mark.parametrize("kind,kw", [("normal", dict(sigma=0.02)), ("laplace", dict(b=0.015)),
                                     ("outlier", dict(sigma=0.02, sigma_out=0.2, p=0.01)), ("uniform", dict(a=0.05))])
@pytest.mark.parametrize("B", [2, 3, 4, 6, 8])
def test_encoder_invariants(kind, kw, B):
    M = (1 << (B - 1)) - 1
    W = datagen.weights(kind, 16, 512, seed=7, **kw)
    G = 128
    k, s, a, b = oracle.encode(W, B, G, "fast")
    ki, si, ai, bi = oracle.encode(W, B, G, "int_clipped")
    assert k.min() >= -M and k.max() <= M  # reserved pattern never emitted
    assert np.all(s > 0)
    for n in range(16):
        for g in range(512 // G):
            sl = slice(g * G, (g + 1) * G)
            assert oracle.shape_margin(float(a[n, g]), float(b[n, g])) > 0  # strictly monotone after rounding
            lev = oracle.levels(B, s[n, g], a[n, g], b[n, g])
            assert np.all(np.diff(lev) > 0)
            e_c = oracle.group_sse(W[n, sl], B, s[n, g], a[n, g], b[n, g], k[n, sl])
            e_i = oracle.group_sse(W[n, sl], B, si[n, g], ai[n, g], bi[n, g], ki[n, sl])
            # the clipped-INT candidates compete first in every search: never worse than clipped INT
            assert e_c <= e_i
            # stored codes are the nearest levels of the stored parameters
            assert np.array_equal(k[n, sl], oracle.assign_group(W[n, sl], B, s[n, g], a[n, g], b[n, g]))
    if B == 2:
        assert np.all(a == ONE) and np.all(b == ZERO)  # shape not identifiable: canonical INT point


def test_zero_group_and_zero_weight():
    W = np.zeros((1, 64), np.float32)
    W[0, 32:] = datagen.weights("normal", 1, 32, seed=8)[0]
    W[0, 40] = 0.0
    for B in (1, 2, 4):
        k, s, a, b = oracle.encode(W, B, 32, "fast")
        assert s[0, 0] == 0.0 and a[0, 0] == ONE and b[0, 0] == ZERO
        assert np.all(k[0, :32] == (1 if B == 1 else 0))
        if B > 1:
            assert k[0, 40] == 0
        codes = oracle.pack(k, B)
        assert np.all(oracle.decode_dense(codes, s, a, b, B, 32, 64)[0, :32] == 0.0)


def test_finite_group_table_soft_pin():
    # Section 3.6 table: G128, 15,360 samples, W2..W6, W8.  The paper's random stream is unnamed, so the
    # pin is the ratio Cubic / clipped INT (<= paper's ratio + 0.01) and exact ties at W2.
    table = {(r[0], int(r[1])): (float(r[2]), float(r[3])) for r in read_table("finite_group_nrmse.txt")}
    n = 15360
    for dist in ("uniform", "gaussian", "laplace"):
        g = datagen.stream(42, "finite-" + dist)
        x = {"uniform": lambda: datagen.uniform_pm(g, n, math.sqrt(3)), "gaussian": lambda: datagen.normal(g, n),
             "laplace": lambda: datagen.laplace(g, n, 1 / math.sqrt(2))}[dist]()
        W = x.astype(np.float32).reshape(n // 128, 128)
        sigma = W.astype(np.float64).std()
        for B in (2, 3, 4, 6, 8):
            res = {}
            for effort in ("reference", "int_clipped"):
                k, s, a, b = oracle.encode(W, B, 128, effort)
                What = oracle.decode_dense(oracle.pack(k, B), s, a, b, B, 128, 128)
                res[effort] = math.sqrt(((W - What) ** 2).mean()) / sigma
            cub, clip = table[(dist, B)]
            assert abs(res["int_clipped"] / clip - 1) < 0.05, (dist, B, res, clip)
            if B == 2:
                assert abs(res["reference"] - res["int_clipped"]) < 1e-3 * clip
            else:
                assert res["reference"] / res["int_clipped"] <= cub / clip + 0.01, (dist, B, res, cub, clip)


# ----------------------------------------------------------------------------- Dynamic A8
def test_quantizer_pins():
    # hand-made rows: max element maps to +-127, exact halves round away from zero, zero row -> zeros
    row = np.zeros((3, 8), np.float32)
    row[0] = [127.0, 0.5, -0.5, 1.5, -1.5, 2.5, 63.5, -126.5]   # d_x = 1 exactly
    row[1] = [0, 0, 0, 0, 0, 0, 0, 0]
    row[2] = [-4.0, 1.0, 2.0, 3.0, 0.25, -0.25, 3.96875, 0.0]
    x = datagen.to_bf16_bits(row)
    assert np.array_equal(datagen.bf16_bits_to_f32(x), row)  # all exactly representable
    x8, dx = oracle.quantize_a8(x)
    assert dx[0] == 1.0
    assert list(x8[0]) == [127, 1, -1, 2, -2, 3, 64, -127]
    assert np.all(x8[1] == 0) and dx[1] == np.float32(np.float32(1e-10) / np.float32(127.0))
    assert x8[2, 0] == -127 and dx[2] == np.float32(4.0) / np.float32(127.0)
    ref = np.float32(row[2]) / dx[2]
    assert list(x8[2]) == [int(math.copysign(math.floor(abs(float(v)) + 0.5), v)) for v in ref]


def test_quantizer_random_rows_max_hits_127():
    x = datagen.activations(32, 512, seed=9, outlier_cols=0.01)
    x8, dx = oracle.quantize_a8(x)
    xf = datagen.bf16_bits_to_f32(x)
    assert np.all(np.abs(x8).max(axis=1) == 127)
    assert np.array_equal(dx, (np.abs(xf).max(axis=1) / np.float32(127.0)).astype(np.float32))
    assert np.all(np.abs(xf - x8 * dx[:, None]) <= 0.5 * dx[:, None] * (1 + 1e-6))


@pytest.mark.parametrize("B", [1, 2, 3, 4, 8])
def test_a8_product_identity_and_bound(B):
    # Eq. continuous-and-carrier-reconstruction: y_A8 equals the plain product of the dequantised
    # activations d_x x8 with the carrier weights s r / 127.
    N, K, G, M = 24, 256, 64, 5
    W = datagen.weights("normal", N, K, seed=12)
    k, s, a, b = oracle.encode(W, B, G, "fast")
    if B > 1:
        k[0, :4] = -(1 << (B - 1))  # reserved pattern contributes zero
    codes = oracle.pack(k, B)
    x = datagen.activations(M, K, seed=13)
    x8, dx = oracle.quantize_a8(x)
    y, P = oracle.gemm_a8(codes, s, a, b, B, G, K, x8, dx, want_partials=True)
    assert np.abs(P).max() <= G * 127 * 127
    car = oracle.carriers_all(B, a, b).astype(np.int64)  # [N, K/G, L]
    kk = oracle.unpack(codes, K, B).astype(np.int64)
    ng = K // G
    r = np.zeros((N, K), np.int64)
    for n in range(N):
        for g in range(ng):
            seg = kk[n, g * G:(g + 1) * G]
            if B == 1:
                r[n, g * G:(g + 1) * G] = np.where(seg > 0, 127, -127)
            else:
                mag = np.where(seg == -(1 << (B - 1)), 0, np.abs(seg))
                r[n, g * G:(g + 1) * G] = np.sign(seg) * car[n, g][mag] * (seg != -(1 << (B - 1)))
    Pref = np.einsum("mgj,ngj->mng", x8.astype(np.int64).reshape(M, ng, G), r.reshape(N, ng, G))
    assert np.array_equal(P, Pref)
    w_a8 = r.reshape(N, ng, G) * (s.astype(np.float64) / 127.0)[:, :, None]
    xt = x8.astype(np.float64) * dx.astype(np.float64)[:, None]
    y2 = xt @ w_a8.reshape(N, K).T
    assert np.allclose(y, y2, rtol=1e-12, atol=1e-18)
    if B <= 2:
        # W1/W2 levels lie on the carrier grid: carrier weights equal continuous weights
        What = oracle.decode_dense(codes, s, a, b, B, G, K)
        assert np.allclose(What, w_a8.reshape(N, K), rtol=1e-7, atol=0)


def test_model_product_matches_dense_matmul():
    N, K, G, M, B = 20, 256, 32, 3, 4
    W = datagen.weights("laplace", N, K, seed=14)
    k, s, a, b = oracle.encode(W, B, G, "fast")
    codes = oracle.pack(k, B)
    x = datagen.activations(M, K, seed=15)
    y = oracle.gemm_model(codes, s, a, b, B, G, K, x)
    What = oracle.decode_dense(codes, s, a, b, B, G, K)
    yref = datagen.bf16_bits_to_f32(x).astype(np.float64) @ What.T
    assert np.allclose(y, yref, rtol=1e-13, atol=1e-18)
    # x . What^T, not x^T or What: a non-square subset distinguishes operands
    ysub = oracle.gemm_model(codes, s, a, b, B, G, K, x, rows=[2, 0], cols=[5, 19, 1])
    assert np.allclose(ysub, yref[[2, 0]][:, [5, 19, 1]], rtol=1e-13)
    # reconstruction is close to the source weights (NRMSE at W4 on Laplace groups ~ 0.1)
    nrmse = math.sqrt(((W - What) ** 2).sum() / (W.astype(np.float64) ** 2).sum())
    assert nrmse < 0.16
    # binary16 activations (Section 5.3: the model-dtype path accepts FP16 or BF16): the same dense matmul on the
    # values numpy's float16 gives those bit patterns; and on values both formats hold exactly the two dtypes agree
    xh = datagen.bf16_bits_to_f32(x).astype(np.float16)
    yh = oracle.gemm_model(codes, s, a, b, B, G, K, xh.view(np.uint16), act="f16")
    assert np.allclose(yh, xh.astype(np.float64) @ What.T, rtol=1e-13, atol=1e-18)
    small = np.round(datagen.bf16_bits_to_f32(x) * 8.0) / 8.0            # multiples of 1/8 below 32: exact in bf16 and fp16
    yb = oracle.gemm_model(codes, s, a, b, B, G, K, datagen.to_bf16_bits(small))
    yf = oracle.gemm_model(codes, s, a, b, B, G, K, small.astype(np.float16).view(np.uint16), act="f16")
    assert np.array_equal(yb, yf)
    x8b, dxb = oracle.quantize_a8(datagen.to_bf16_bits(small))
    x8f, dxf = oracle.quantize_a8(small.astype(np.float16).view(np.uint16), act="f16")
    assert np.array_equal(x8b, x8f) and np.array_equal(dxb, dxf)
