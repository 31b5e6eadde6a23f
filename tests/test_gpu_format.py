"""GPU parity of the format pieces against the oracle: packing, layout round trip, levels,
carriers, dense decode, activation quantiser, integer partials.  Integer/byte results bit-exact."""
import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2608_06763_b200 as cq
from util import Case, encoded_case, logical_case, x_to_device

pytestmark = pytest.mark.gpu

ALL_B = [1, 2, 3, 4, 5, 6, 7, 8]


@pytest.mark.parametrize("B", ALL_B)
def test_pack_codes_matches_oracle_bitstream(B):
    k, _, _, _ = datagen.logical_quantized(5, 328, B, 8, seed=20 + B)  # 328*B/8 ragged for odd B? 328 = 8*41
    k = k[:, :321] if B % 2 else k  # odd widths: K*B not a multiple of 8 -> row tail
    k = np.ascontiguousarray(k)
    if B > 1:
        k[0, :3] = -(1 << (B - 1))  # reserved pattern survives packing
    got = cq.cq_pack_codes(torch.from_numpy(k).cuda(), B).cpu().numpy()
    assert np.array_equal(got, oracle.pack(k, B))


@pytest.mark.parametrize("G", [32, 64, 128, 256, 512])
@pytest.mark.parametrize("B", ALL_B)
def test_repack_unpack_roundtrip_bit_exact(B, G):
    N, K = 200, 384 if G <= 128 else 1024  # N not a multiple of 128: padded rows
    c = logical_case(N, K, B, G, seed=30 + B)
    if B > 1:
        c.k[3, 5:9] = -(1 << (B - 1))
        c = Case(c.k, c.s, c.a, c.b, B, G)
    codes, s, a, b = cq.cq_unpack(c.pw)
    assert np.array_equal(codes.cpu().numpy(), c.codes)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), c.s.view(np.uint32))
    assert np.array_equal(a.cpu().numpy().view(np.uint16), np.ascontiguousarray(c.a).view(np.uint16))
    assert np.array_equal(b.cpu().numpy().view(np.uint16), np.ascontiguousarray(c.b).view(np.uint16))


@pytest.mark.parametrize("B", ALL_B)
def test_levels_within_1e6_relative(B):
    c = encoded_case("laplace", 96, 512, B, 64, seed=40 + B, b=0.015)
    got = cq.cq_decode_levels(c.pw).cpu().numpy().astype(np.float64)
    ref = oracle.levels_all(B, c.s, c.a, c.b)
    assert got.shape == ref.shape
    denom = np.maximum(np.abs(ref), 1e-30)
    assert np.all(np.abs(got - ref) <= 1e-6 * denom + 1e-38), float((np.abs(got - ref) / denom).max())


@pytest.mark.parametrize("B", [3, 4, 6, 8])
def test_levels_random_admissible_shapes(B):
    c = logical_case(128, 256, B, 32, seed=50 + B)  # a in [0.5, 1], b in [-0.3, 0]
    got = cq.cq_decode_levels(c.pw).cpu().numpy().astype(np.float64)
    ref = oracle.levels_all(B, c.s, c.a, c.b)
    assert np.all(np.abs(got - ref) <= 1e-6 * np.abs(ref))


@pytest.mark.parametrize("B", ALL_B)
def test_carriers_bit_exact(B):
    c = logical_case(128, 512, B, 32, seed=60 + B)
    got = cq.cq_decode_carriers(c.pw).cpu().numpy()
    assert np.array_equal(got, oracle.carriers_all(B, c.a, c.b))
    c2 = encoded_case("normal", 64, 256, B, 128, seed=61 + B)
    assert np.array_equal(cq.cq_decode_carriers(c2.pw).cpu().numpy(), oracle.carriers_all(B, c2.a, c2.b))


@pytest.mark.parametrize("B", ALL_B)
def test_dense_decode_sign_and_magnitude(B):
    c = logical_case(130, 256, B, 64, seed=70 + B)
    if B > 1:
        c.k[1, :7] = -(1 << (B - 1))
        c = Case(c.k, c.s, c.a, c.b, B, 64)
    got = cq.cq_decode_weights(c.pw).cpu().numpy().astype(np.float64)
    ref = oracle.decode_dense(c.codes, c.s, c.a, c.b, B, 64, c.K)
    assert np.array_equal(np.sign(got), np.sign(ref))
    assert np.all(np.abs(got - ref) <= 1e-6 * np.abs(ref))


def test_quantizer_bit_exact():
    rows = [datagen.activations(48, 1000, seed=80, outlier_cols=0.01)]
    special = np.zeros((4, 1000), np.float32)
    special[0, :8] = [127.0, 0.5, -0.5, 1.5, -1.5, 2.5, 63.5, -126.5]
    special[2, :4] = [1e-20, -3e-21, 0, 2e-30]  # below the epsilon safeguard
    special[3] = np.linspace(-3, 3, 1000)
    rows.append(datagen.to_bf16_bits(special))
    x = np.concatenate(rows, axis=0)
    x8, dx = cq.cq_quantize_a8(x_to_device(x))
    rx8, rdx = oracle.quantize_a8(x)
    assert np.array_equal(dx.cpu().numpy().view(np.uint32), rdx.view(np.uint32))
    assert np.array_equal(x8.cpu().numpy(), rx8)


@pytest.mark.parametrize("B", [1, 2, 3, 4, 6, 8])
def test_a8_integer_partials_bit_exact(B):
    c = encoded_case("normal", 40, 256, B, 64, seed=90 + B)
    x = datagen.activations(5, 256, seed=91, outlier_cols=0.02)
    rx8, rdx = oracle.quantize_a8(x)
    P = cq.cq_debug_a8_partials(c.pw, torch.from_numpy(rx8).cuda()).cpu().numpy()
    _, Pref = oracle.gemm_a8(c.codes, c.s, c.a, c.b, B, 64, c.K, rx8, rdx, want_partials=True)
    assert np.array_equal(P, Pref)


@pytest.mark.parametrize("G", [256, 512])
@pytest.mark.parametrize("B", [2, 5, 8])
def test_wide_groups_levels_carriers_partials(B, G):
    # group sizes of the paper's own kernel measurements
    c = logical_case(72, 1024, B, G, seed=95 + B)
    c.k[3, 300:310] = -(1 << (B - 1))
    c = Case(c.k, c.s, c.a, c.b, B, G)
    ref = oracle.levels_all(B, c.s, c.a, c.b)
    got = cq.cq_decode_levels(c.pw).cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref) <= 1e-6 * np.abs(ref))
    assert np.array_equal(cq.cq_decode_carriers(c.pw).cpu().numpy(), oracle.carriers_all(B, c.a, c.b))
    W = cq.cq_decode_weights(c.pw).cpu().numpy().astype(np.float64)
    Wr = oracle.decode_dense(c.codes, c.s, c.a, c.b, B, G, c.K)
    assert np.array_equal(np.sign(W), np.sign(Wr)) and np.all(np.abs(W - Wr) <= 1e-6 * np.abs(Wr))
    x = datagen.activations(3, 1024, seed=96)
    rx8, rdx = oracle.quantize_a8(x)
    P = cq.cq_debug_a8_partials(c.pw, torch.from_numpy(rx8).cuda()).cpu().numpy()
    _, Pref = oracle.gemm_a8(c.codes, c.s, c.a, c.b, B, G, c.K, rx8, rdx, want_partials=True)
    assert np.array_equal(P, Pref) and np.abs(P).max() <= G * 127 * 127
