"""Tests that go through cq_gemm itself (the kernels the product runs, not the side kernels written for
clarity) on inputs whose result is known exactly or almost exactly, so that one wrong carrier byte, a
swapped k position or an off-by-one table entry fails:

  - Dynamic A8 (Eq. a8-output) on integer activations with max |x| = 127 (d_x = 1 exactly, x8 = x) and
    scales 127 * 2^-j (d_x s_g / 127 is a power of two): every group partial and every fp32 sum is an
    exactly representable number, so y must equal the oracle's y rounded to bf16 BIT FOR BIT, on the
    INT8 mma.sync kernel (M <= 16) and on the tcgen05 INT8 kernel (M > 16, with and without split-K);
  - model dtype on one-hot activations: y[m, n] is the decoded weight of one (n, k) itself, compared with
    the oracle's level within the fp16 / bf16 rounding of the path, for every k position of a tile, on the
    one- and two-token kernel, the MMA kernel and the tcgen05 kernel, including shapes at the edges of the
    admissible domain (Eq. monotonicity) where the cubic's terms cancel.
"""
import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2608_06763_b200 as cq
from util import Case, check_y, x_to_device, y_to_numpy

pytestmark = pytest.mark.gpu

# (a, b) pairs: the integer grid, interior fits, and the edges of the strictly monotone domain
# q'(t) = a + 2 b t + 3 (1 - a - b) t^2 > 0 on [0, 1]: a -> 0+, the corners of a fitter's grid, refined shapes
# with |b| > 1, and one whose derivative almost vanishes at t = 1
EDGE_SHAPES = [(1.0, 0.0), (0.7, -0.2), (0.2, 0.2), (1.2, -1.0), (0.05, 0.1), (2.0, -2.5), (2.9, -2.85), (0.36, -0.73), (0.3, 1.5)]


def edge_case(N, K, B, G, seed, scales=None):
    """Uniform random codes over the whole range (a few reserved patterns), shapes cycling through EDGE_SHAPES."""
    g = datagen.stream(seed, f"edge-B{B}-G{G}")
    Mx = (1 << (B - 1)) - 1
    if B == 1:
        k = np.where(datagen.uniform01(g, N * K) < 0.5, -1, 1).astype(np.int8).reshape(N, K)
    else:
        k = (np.floor(datagen.uniform01(g, N * K) * (2 * Mx + 1)) - Mx).astype(np.int8).reshape(N, K)
        k[3, 5:9] = -(1 << (B - 1))          # reserved pattern decodes to zero
        k[N - 1, K - 1] = -(1 << (B - 1))
    ng = K // G
    idx = (np.arange(N * ng) * 7 + seed) % len(EDGE_SHAPES)
    a = np.array([EDGE_SHAPES[i][0] for i in idx], np.float16).reshape(N, ng)
    b = np.array([EDGE_SHAPES[i][1] for i in idx], np.float16).reshape(N, ng)
    for av, bv in zip(a.ravel()[:len(EDGE_SHAPES)], b.ravel()[:len(EDGE_SHAPES)]):
        assert oracle.shape_margin(float(av), float(bv)) > 0.0     # all admissible after the fp16 rounding
    if scales is None:
        s = (0.03 + 0.06 * datagen.uniform01(g, N * ng)).astype(np.float32).reshape(N, ng)
    else:
        s = np.asarray(scales, np.float32).reshape(N, ng)
    return Case(k, s, a, b, B, G)


def integer_activations(M, K, G, nnz, seed):
    """Rows of small integers: nnz entries of +-1, +-2 per group, one +-127 per row (so d_x = 1)."""
    g = datagen.stream(seed, "int-x")
    x = np.zeros((M, K), np.float32)
    for m in range(M):
        for gi in range(K // G):
            pos = g.choice(G, nnz, replace=False) + gi * G
            x[m, pos] = g.choice(np.array([-2.0, -1.0, 1.0, 2.0]), nnz)
        x[m, int(g.integers(0, K))] = 127.0 if m % 2 == 0 else -127.0
    bits = datagen.to_bf16_bits(x)
    assert np.array_equal(datagen.bf16_bits_to_f32(bits), x)
    return bits


def a8_exact(c, xb):
    x8, dx = oracle.quantize_a8(xb)
    assert np.all(dx == 1.0) and np.array_equal(x8.astype(np.float32), datagen.bf16_bits_to_f32(xb))
    ref = oracle.gemm_a8(c.codes, c.s, c.a, c.b, c.B, c.G, c.K, x8, dx)
    want = datagen.to_bf16_bits(ref.astype(np.float32))
    assert np.array_equal(ref.astype(np.float32).astype(np.float64), ref)   # the exact result fits fp32: nothing rounds before the bf16 cast
    ws = torch.zeros(cq.cq_workspace_bytes(c.B, c.G, xb.shape[0], c.N, c.K, cq.CQ_DYN_A8), dtype=torch.uint8, device="cuda")
    y = cq.cq_gemm(c.pw, x_to_device(xb), cq.CQ_DYN_A8, ws)
    assert cq.cq_gemm_status(ws) == 0
    got = y.view(torch.int16).cpu().numpy().view(np.uint16)
    bad = np.argwhere(got != want)
    assert bad.size == 0, (len(bad), bad[:5], datagen.bf16_bits_to_f32(got)[tuple(bad[0])], ref[tuple(bad[0])])


def power_of_two_scales(n, seed, jmax):
    g = datagen.stream(seed, "pow2-scales")
    return (127.0 * np.exp2(-g.integers(0, jmax + 1, n).astype(np.float64))).astype(np.float32)


@pytest.mark.parametrize("M", [1, 5, 16])
@pytest.mark.parametrize("G", [32, 64, 128])
@pytest.mark.parametrize("B", [1, 2, 3, 4, 5, 6, 7, 8])
def test_a8_small_m_kernel_bit_exact(B, G, M):
    N, K = 200, 4 * G if G >= 64 else 8 * G
    c = edge_case(N, K, B, G, seed=500 + B, scales=power_of_two_scales(N * (K // G), 510 + B, 1))
    a8_exact(c, integer_activations(M, K, G, 8, seed=520 + M))


@pytest.mark.parametrize("M,K", [(40, 512), (150, 512), (300, 512), (100, 2048), (200, 2048)])
@pytest.mark.parametrize("G", [32, 64, 128])
@pytest.mark.parametrize("B", [1, 2, 3, 4, 5, 6, 7, 8])
def test_a8_tcgen05_kernel_bit_exact(B, G, M, K):
    # K = 2048 with few output tiles cuts K into slices (the last CTA of a tile adds them); K = 512 runs without
    N = 200
    plan = cq.cq_debug_gemm_plan(B, G, M, N, K, cq.CQ_DYN_A8)
    assert (plan["stream_k_ctas"] > plan["stream_k_tiles"]) == (K == 2048), plan
    nnz = 8 if K == 512 else 2
    c = edge_case(N, K, B, G, seed=530 + B, scales=power_of_two_scales(N * (K // G), 540 + B, 1 if K == 512 else 0))
    a8_exact(c, integer_activations(M, K, G, nnz, seed=550 + M))


def one_hot_check(c, M, positions, what):
    """x[m] = e_{positions[m]}: y[m, n] must be the decoded weight (n, positions[m])."""
    x = np.zeros((M, c.K), np.float32)
    x[np.arange(M), positions] = 1.0
    y = y_to_numpy(cq.cq_gemm(c.pw, x_to_device(datagen.to_bf16_bits(x)), cq.CQ_MODEL_DTYPE))
    What = oracle.decode_dense(c.codes, c.s, c.a, c.b, c.B, c.G, c.K)            # [N, K] fp64
    want = What[:, positions].T                                                  # [M, N]
    scale = np.repeat(c.s, c.G, axis=1)[:, positions].T.astype(np.float64)
    # bf16 output rounding (2^-9 relative) plus the fp16 level arithmetic (a few 2^-11 of the group scale)
    tol = 2.0 ** -7 * np.abs(want) + 2.0 ** -9 * scale
    err = np.abs(y - want)
    bad = np.argwhere(err > tol)
    assert bad.size == 0, (what, len(bad), bad[:5], y[tuple(bad[0])], want[tuple(bad[0])])
    assert np.all(y[want == 0.0] == 0.0)                                         # code 0 and the reserved pattern


@pytest.mark.parametrize("G", [32, 128])
@pytest.mark.parametrize("B", [1, 2, 3, 4, 5, 6, 7, 8])
def test_model_dtype_one_hot_every_k_position(B, G):
    N, K = 136, 256                      # two 128-wide tiles; N ragged against the 128-row tile
    c = edge_case(N, K, B, G, seed=560 + B)
    g = datagen.stream(561, "positions")
    for M in (1, 2, 7, 16):             # the one- and two-token kernel, then the MMA kernel with one and two token blocks
        for rep in range(2 if M <= 2 else 1):
            one_hot_check(c, M, g.choice(K, M, replace=False), f"B={B} G={G} M={M}")
    one_hot_check(c, 16, np.arange(16) * 16 + 5, f"B={B} G={G} strided")
    one_hot_check(c, K, g.permutation(K), f"B={B} G={G} tcgen05 all positions")   # M = 256: the tcgen05 kernel, every k


@pytest.mark.parametrize("mode", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
@pytest.mark.parametrize("M", [1, 2, 8, 64])
@pytest.mark.parametrize("B", [3, 4, 5, 6, 8])
def test_edge_shapes_within_tolerance(B, M, mode):
    # the benchmark spec's tolerance on shapes at the edge of the admissible domain, dense random activations
    N, K, G = 200, 1024, 128
    c = edge_case(N, K, B, G, seed=570 + B)
    xb = datagen.activations(M, K, seed=571, outlier_cols=0.01)
    y = y_to_numpy(cq.cq_gemm(c.pw, x_to_device(xb), mode))
    if mode == cq.CQ_MODEL_DTYPE:
        ref = oracle.gemm_model(c.codes, c.s, c.a, c.b, B, G, K, xb)
    else:
        x8, dx = oracle.quantize_a8(xb)
        ref = oracle.gemm_a8(c.codes, c.s, c.a, c.b, B, G, K, x8, dx)
    check_y(y, ref, f"edge shapes B={B} M={M} mode={mode}")
