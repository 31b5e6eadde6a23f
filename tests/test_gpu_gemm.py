"""GPU parity of cq_gemm against the oracle at sizes the oracle finishes in seconds: every width,
every group size, both modes, M across the small-M / large-M boundary, ragged N and K."""
import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2608_06763_b200 as cq
from util import Case, check_y, encoded_case, logical_case, x_to_device, y_to_numpy

pytestmark = pytest.mark.gpu

ALL_B = [1, 2, 3, 4, 5, 6, 7, 8]


def run_both(c, x_bits, mode):
    y = y_to_numpy(cq.cq_gemm(c.pw, x_to_device(x_bits), mode))
    if mode == cq.CQ_MODEL_DTYPE:
        ref = oracle.gemm_model(c.codes, c.s, c.a, c.b, c.B, c.G, c.K, x_bits)
    else:
        x8, dx = oracle.quantize_a8(x_bits)
        ref = oracle.gemm_a8(c.codes, c.s, c.a, c.b, c.B, c.G, c.K, x8, dx)
    return y, ref


@pytest.mark.parametrize("mode", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
@pytest.mark.parametrize("G", [32, 64, 128])
@pytest.mark.parametrize("B", ALL_B)
def test_gemv_m1_all_widths_and_groups(B, G, mode):
    c = encoded_case("laplace", 384, 1024, B, G, seed=100 + B, b=0.015)
    x = datagen.activations(1, 1024, seed=101)
    y, ref = run_both(c, x, mode)
    check_y(y, ref, f"B={B} G={G} mode={mode}")


@pytest.mark.parametrize("mode", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
@pytest.mark.parametrize("M", [1, 3, 8, 9, 16])
def test_small_m_rows(M, mode):
    c = encoded_case("outlier", 256, 2048, 4, 128, seed=110, sigma=0.02, sigma_out=0.2, p=0.001)
    x = datagen.activations(M, 2048, seed=111, outlier_cols=0.01)
    y, ref = run_both(c, x, mode)
    check_y(y, ref, f"M={M} mode={mode}")


@pytest.mark.parametrize("mode", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
@pytest.mark.parametrize("B", [2, 3, 4, 8])
def test_ragged_shapes_and_reserved_codes(B, mode):
    # N and K not multiples of the 128 tile, K not a multiple of 8 elements per row is not allowed by
    # K % G == 0, so the ragged K case is K = 3 * 32 + 128 ... = 224 (G = 32)
    N, K, G = 200, 224, 32
    c = logical_case(N, K, B, G, seed=120 + B)
    c.k[7, 10:20] = -(1 << (B - 1))  # reserved pattern decodes to zero
    c.k[150, :] = 0
    c.s[9, 2] = 0.0                   # all-zero group
    c = Case(c.k, c.s, c.a, c.b, B, G)
    x = datagen.activations(5, K, seed=121)
    y, ref = run_both(c, x, mode)
    check_y(y, ref, f"ragged B={B} mode={mode}")
    assert np.all(y[:, 150] == 0.0)


@pytest.mark.parametrize("mode", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
def test_extreme_activation_magnitudes(mode):
    # rows with huge and tiny magnitudes: the per-row scaling must neither overflow nor flush
    c = encoded_case("normal", 128, 512, 4, 128, seed=130)
    x = datagen.bf16_bits_to_f32(datagen.activations(4, 512, seed=131)).copy()
    x[0] *= 3.0e4
    x[1] *= 1.0e-6
    x[2, :] = 0.0
    x[3, 17] = 5.0e5
    xb = datagen.to_bf16_bits(x)
    y, ref = run_both(c, xb, mode)
    for m in range(4):
        if m == 2:
            assert np.all(y[m] == 0)
        else:
            check_y(y[m:m + 1], ref[m:m + 1], f"row {m} mode={mode}")


@pytest.mark.parametrize("mode", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
@pytest.mark.parametrize("M", [17, 64, 129, 300])
@pytest.mark.parametrize("B", [3, 4, 8])
def test_large_m_rows(B, M, mode):
    c = encoded_case("normal", 256, 1024, B, 128, seed=140 + B, sigma=0.015)
    x = datagen.activations(M, 1024, seed=141, outlier_cols=0.01)
    y, ref = run_both(c, x, mode)
    check_y(y, ref, f"B={B} M={M} mode={mode}")


def test_repeatable_bitwise_and_workspace_reuse():
    c = encoded_case("normal", 512, 4096, 4, 128, seed=150)
    x = x_to_device(datagen.activations(4, 4096, seed=151))
    ws = torch.zeros(cq.cq_workspace_bytes(4, 128, 4, 512, 4096, 0), dtype=torch.uint8, device="cuda")
    y1 = cq.cq_gemm(c.pw, x, 0, ws).clone()
    y2 = cq.cq_gemm(c.pw, x, 0, ws).clone()
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))  # fixed split-K order: deterministic


@pytest.mark.parametrize("G", [32, 64, 128])
@pytest.mark.parametrize("B", ALL_B)
def test_tensor_core_gemm_all_widths_and_groups(B, G):
    # M = 40 runs the tcgen05 path with a 64-token tile; ragged N and K, reserved codes, a zero group
    N, K = 200, 352 if G == 32 else 384
    c = logical_case(N, K, B, G, seed=160 + B)
    if B > 1:
        c.k[5, 3:40] = -(1 << (B - 1))
    c.s[17, 1] = 0.0
    c = Case(c.k, c.s, c.a, c.b, B, G)
    x = datagen.activations(40, K, seed=161)
    y, ref = run_both(c, x, cq.CQ_MODEL_DTYPE)
    check_y(y, ref, f"tc B={B} G={G}")


@pytest.mark.parametrize("M", [513, 700])
def test_tensor_core_gemm_wide_token_tile(M):
    # more than 512 rows: 256-token tiles, last tile ragged
    c = encoded_case("normal", 384, 1024, 4, 128, seed=170, sigma=0.015)
    x = datagen.activations(M, 1024, seed=171)
    y, ref = run_both(c, x, cq.CQ_MODEL_DTYPE)
    check_y(y, ref, f"tc M={M}")
    ws = torch.zeros(cq.cq_workspace_bytes(4, 128, M, 384, 1024, 0), dtype=torch.uint8, device="cuda")
    cq.cq_gemm(c.pw, x_to_device(x), 0, ws)
    assert cq.cq_gemm_status(ws) == 0


# Stream-K: output tiles shared by several CTAs (partial tiles through the workspace, added in K order by the
# last CTA to arrive).  (N, K, M, runs cross tiles): few tiles, each cut into many runs; one tile, ragged in N, K
# and M; more tiles than SMs, so that whole-tile CTAs and runs share a launch; a 512-token tile with a ragged last
# tile; a last round of 76 tiles shared by one run per SM, so that runs cross from one tile into the next (the
# kernel of cq_gemm_tc_sk.cu).
STREAM_K_SHAPES = [(256, 8192, 40, False), (100, 4096 + 128, 33, False), (128 * 150, 4096, 40, False),
                   (384, 8192, 700, False), (128 * (148 + 76), 4096, 20, True)]


@pytest.mark.parametrize("act", ["bf16", "f16"])
@pytest.mark.parametrize("N,K,M,crossing", STREAM_K_SHAPES)
def test_tensor_core_gemm_stream_k(N, K, M, crossing, act):
    B, G = (4, 128) if N != 100 else (3, 64)
    plan = cq.cq_debug_gemm_plan(B, G, M, N, K)
    assert plan["stream_k_ctas"] > plan["stream_k_tiles"] > 0, plan   # the shape does share tiles between CTAs
    if torch.cuda.get_device_properties(0).multi_processor_count == 148:
        assert plan["runs_cross_tiles"] == crossing, plan
    if N > 128 * 148:
        assert plan["whole_tile_ctas"] > 0, plan
    c = logical_case(N, K, B, G, seed=180 + M)
    x = datagen.activations(M, K, seed=181, outlier_cols=0.01)      # bf16 bit patterns
    if act == "f16":
        x = datagen.bf16_bits_to_f32(x).astype(np.float16).view(np.uint16)
        xd = torch.from_numpy(x.view(np.float16)).cuda()
    else:
        xd = x_to_device(x)
    ws = torch.zeros(cq.cq_workspace_bytes(B, G, M, N, K, 0), dtype=torch.uint8, device="cuda")
    y1 = cq.cq_gemm(c.pw, xd, 0, ws).clone()
    assert cq.cq_gemm_status(ws) == 0
    y2 = cq.cq_gemm(c.pw, xd, 0, ws).clone()          # the counters were left at zero; fixed order of addition
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))
    ref = oracle.gemm_model(c.codes, c.s, c.a, c.b, c.B, c.G, c.K, x, act=act)
    yn = y_to_numpy(y1) if act == "bf16" else y1.cpu().numpy().astype(np.float64)
    check_y(yn, ref, f"stream-K N={N} K={K} M={M} {act}")


@pytest.mark.parametrize("G", [32, 64, 128])
@pytest.mark.parametrize("B", ALL_B)
def test_tensor_core_a8_gemm_all_widths_and_groups(B, G):
    # M = 150 runs the tcgen05 INT8 path (two token tiles, the last ragged); ragged N and K,
    # reserved codes, a zero group, activation outlier columns
    N, K = 200, 352 if G == 32 else 384
    c = logical_case(N, K, B, G, seed=180 + B)
    if B > 1:
        c.k[5, 3:40] = -(1 << (B - 1))
    c.s[17, 1] = 0.0
    c = Case(c.k, c.s, c.a, c.b, B, G)
    x = datagen.activations(150, K, seed=181, outlier_cols=0.02)
    y, ref = run_both(c, x, cq.CQ_DYN_A8)
    check_y(y, ref, f"a8 tc B={B} G={G}")


@pytest.mark.parametrize("mode", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
@pytest.mark.parametrize("M", [1, 16, 64, 300])
@pytest.mark.parametrize("B,G", [(2, 512), (5, 512), (8, 256), (4, 256)])
def test_wide_groups_all_paths(B, G, M, mode):
    # G = 256 / 512 (the group sizes of the paper's H200 measurements) through every kernel
    c = encoded_case("normal", 200, 1024, B, G, seed=190 + B)
    x = datagen.activations(M, 1024, seed=191, outlier_cols=0.01)
    y, ref = run_both(c, x, mode)
    check_y(y, ref, f"G={G} B={B} M={M} mode={mode}")


@pytest.mark.parametrize("G", [64, 128])
@pytest.mark.parametrize("M", [40, 100, 128, 200])
def test_a8_gemm_token_tiles_and_split_k(M, G):
    # few output tiles and a long K: the INT8 tcgen05 path picks its token tile from M (64 / 128 / 256,
    # capped by the group count) and cuts K into slices combined in slice order; two calls on one
    # workspace must agree bit for bit (arrival counters are left cleared)
    N, K, B = 200, 2048, 4
    plan = cq.cq_debug_gemm_plan(B, G, M, N, K, cq.CQ_DYN_A8)
    assert plan["stream_k_ctas"] > plan["stream_k_tiles"] > 0, plan     # the tiles are cut into slices
    c = logical_case(N, K, B, G, seed=190 + M)
    c.k[7, 100:140] = -(1 << (B - 1))
    c = Case(c.k, c.s, c.a, c.b, B, G)
    x = datagen.activations(M, K, seed=191, outlier_cols=0.01)
    y, ref = run_both(c, x, cq.CQ_DYN_A8)
    check_y(y, ref, f"a8 split-K M={M} G={G}")
    ws = torch.zeros(cq.cq_workspace_bytes(B, G, M, N, K, 1), dtype=torch.uint8, device="cuda")
    xd = x_to_device(x)
    y1 = cq.cq_gemm(c.pw, xd, 1, ws).clone()
    y2 = cq.cq_gemm(c.pw, xd, 1, ws).clone()
    assert cq.cq_gemm_status(ws) == 0
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))
    assert np.array_equal(y_to_numpy(y1), y)


def test_random_shapes_both_modes():
    # seeded shape fuzz: ragged N and K, every width and group size, M on both sides of every dispatch
    # boundary (16 | 17, token tiles, split-K on / off), a few reserved codes in every case
    rng = np.random.default_rng(20240607)
    Ms = [1, 2, 5, 8, 9, 16, 17, 31, 33, 64, 65, 127, 130, 257, 600]
    for trial in range(28):
        B = int(rng.integers(1, 9))
        G = int(rng.choice([32, 64, 128, 256, 512]))
        K = G * int(rng.integers(1, max(2, 2304 // G)))
        N = int(rng.integers(1, 420))
        M = int(rng.choice(Ms))
        mode = int(rng.integers(0, 2))
        c = logical_case(N, K, B, G, seed=300 + trial)
        if B > 1:
            c.k[int(rng.integers(0, N)), int(rng.integers(0, K))] = -(1 << (B - 1))
            c = Case(c.k, c.s, c.a, c.b, B, G)
        x = datagen.activations(M, K, seed=400 + trial, outlier_cols=0.01 if trial % 3 == 0 else 0.0)
        y, ref = run_both(c, x, mode)
        check_y(y, ref, f"fuzz trial={trial} B={B} G={G} N={N} K={K} M={M} mode={mode}")


def test_bounded_wait_gives_up_and_is_reported():
    # the failure path of the pipelined kernels without any failure: one wait on a barrier nobody arrives
    # on, with nothing in flight, runs out after about a millisecond; the kernel ends normally, the status
    # word says CQ_ERR_TIMEOUT, and the same workspace serves a correct product once it is re-initialised
    c = logical_case(256, 512, 4, 128, seed=700)
    x = x_to_device(datagen.activations(40, 512, seed=701))
    ws = torch.zeros(cq.cq_workspace_bytes(4, 128, 40, 256, 512, 0), dtype=torch.uint8, device="cuda")
    assert cq.cq_gemm_status(ws) == 0
    cq.cq_debug_wait_timeout(ws, 2_000_000)
    assert cq.cq_gemm_status(ws) == -7 and cq.cq_status_string(-7) == "CQ_ERR_TIMEOUT"
    assert cq.cq_gemm_status(ws) == -7            # sticky until the workspace is re-initialised
    cq.cq_workspace_init(ws)
    assert cq.cq_gemm_status(ws) == 0
    y = y_to_numpy(cq.cq_gemm(c.pw, x, cq.CQ_MODEL_DTYPE, ws))
    assert cq.cq_gemm_status(ws) == 0
    xb = x.view(torch.int16).cpu().numpy().view(np.uint16)
    check_y(y, oracle.gemm_model(c.codes, c.s, c.a, c.b, 4, 128, 512, xb), "after a reported timeout")
