"""binary16 activations (Section 5.3: the model-dtype path accepts FP16 or BF16 activations) through every
kernel of cq_gemm, against the oracle evaluated on the same binary16 values."""
import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2608_06763_b200 as cq
from util import Case, check_y, encoded_case, logical_case

pytestmark = pytest.mark.gpu


def half_activations(M, K, seed, scale=1.0, outlier_cols=0.0):
    x = datagen.bf16_bits_to_f32(datagen.activations(M, K, seed=seed, outlier_cols=outlier_cols)).astype(np.float64) * scale
    # perturb below bf16 precision so that the values really use binary16's 11-bit significand
    x = x * (1.0 + 2.0 ** -10 * datagen.uniform01(datagen.stream(seed, "f16-jitter"), M * K).reshape(M, K))
    return x.astype(np.float16)


def run(c, xh, mode):
    y = cq.cq_gemm(c.pw, torch.from_numpy(xh).cuda(), mode)
    assert y.dtype == torch.float16
    bits = xh.view(np.uint16)
    if mode == cq.CQ_MODEL_DTYPE:
        ref = oracle.gemm_model(c.codes, c.s, c.a, c.b, c.B, c.G, c.K, bits, act="f16")
    else:
        x8, dx = oracle.quantize_a8(bits, act="f16")
        ref = oracle.gemm_a8(c.codes, c.s, c.a, c.b, c.B, c.G, c.K, x8, dx)
    return y.float().cpu().numpy().astype(np.float64), ref


@pytest.mark.parametrize("mode", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
@pytest.mark.parametrize("M", [1, 2, 7, 16, 40, 300, 600])
@pytest.mark.parametrize("B,G", [(1, 128), (2, 64), (3, 128), (4, 128), (4, 32), (6, 64), (8, 128), (5, 512)])
def test_f16_activations_all_kernels(B, G, M, mode):
    c = logical_case(200, 1024, B, G, seed=800 + B)
    if B > 1:
        c.k[5, 3:40] = -(1 << (B - 1))
        c = Case(c.k, c.s, c.a, c.b, B, G)
    xh = half_activations(M, 1024, seed=801 + M, outlier_cols=0.01)
    y, ref = run(c, xh, mode)
    check_y(y, ref, f"f16 B={B} G={G} M={M} mode={mode}")


def test_f16_output_is_finer_than_bf16():
    # the binary16 result carries 11 significant bits: the same product is closer to the oracle than a bf16 one can be
    c = encoded_case("normal", 256, 2048, 4, 128, seed=810)
    xh = half_activations(8, 2048, seed=811)
    y, ref = run(c, xh, cq.CQ_MODEL_DTYPE)
    assert np.linalg.norm(y - ref) / np.linalg.norm(ref) < 1.2e-3        # bf16 output rounding alone costs 1.6e-3


@pytest.mark.parametrize("scale", [1.0, 3.0e3, 1.0e-5])
def test_f16_extreme_magnitudes_and_quantiser_bit_exact(scale):
    # rows near the top of the binary16 range and rows of subnormals: the per-row rescaling keeps the products exact,
    # and the quantiser matches the oracle bit for bit
    c = encoded_case("normal", 128, 512, 4, 128, seed=820)
    xh = half_activations(4, 512, seed=821, scale=scale)
    xh[2, :] = 0.0
    for mode in (cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8):
        y, ref = run(c, xh, mode)
        assert np.all(y[2] == 0)
        for m in (0, 1, 3):
            check_y(y[m:m + 1], ref[m:m + 1], f"f16 scale={scale} row {m} mode={mode}")
    x8, dx = cq.cq_quantize_a8(torch.from_numpy(xh).cuda())
    x8o, dxo = oracle.quantize_a8(xh.view(np.uint16), act="f16")
    assert np.array_equal(x8.cpu().numpy(), x8o) and np.array_equal(dx.cpu().numpy(), dxo)
