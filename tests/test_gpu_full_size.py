"""Parity at the full sizes of the five benchmark configurations, in the launch configuration the
benchmark times (same entry point, same dispatch), on outputs the oracle computes one by one:
whole y where that is cheap, otherwise a seeded sample of activation rows x output channels.

Weights of configuration 1 are fitted by the oracle encoder; the larger tensors use the seeded
already-quantised recipe of datagen (running the fitter on 10^8..10^9 weights takes too long), which
the library packs itself while the oracle packs the sampled rows with its own packer."""
import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2608_06763_b200 as cq
from util import Case, check_y, x_to_device, y_to_numpy

pytestmark = pytest.mark.gpu


def sampled_reference(k_rows, s_rows, a_rows, b_rows, B, G, K, x_bits, mode, rows=None):
    """Oracle y[rows, sampled channels] from the sampled channels' logical codes and parameters."""
    codes = oracle.pack(np.ascontiguousarray(k_rows), B)
    if mode == cq.CQ_MODEL_DTYPE:
        return oracle.gemm_model(codes, s_rows, a_rows, b_rows, B, G, K, x_bits, rows=rows)
    x8, dx = oracle.quantize_a8(x_bits)
    return oracle.gemm_a8(codes, s_rows, a_rows, b_rows, B, G, K, x8, dx, rows=rows)


def test_config1_w4_g128_gemv_oracle_encoded():
    # 4096 x 4096, N(0, 0.02^2) seed 0, fitted by the oracle encoder, x ~ N(0,1), M = 1
    N = K = 4096
    W = datagen.weights("normal", N, K, seed=0, sigma=0.02)
    k, s, a, b = oracle.encode(W, 4, 128, "fast")
    c = Case(k, s, a, b, 4, 128)
    xb = datagen.activations(1, K, seed=0)
    y = y_to_numpy(cq.cq_gemm(c.pw, x_to_device(xb), cq.CQ_MODEL_DTYPE))
    ref = oracle.gemm_model(c.codes, s, a, b, 4, 128, K, xb)
    check_y(y, ref, "config 1")
    # the quantised product stays close to the unquantised one (W4 on Gaussian groups: NRMSE ~ 0.09)
    exact = datagen.bf16_bits_to_f32(xb).astype(np.float64) @ W.astype(np.float64).T
    assert np.linalg.norm(ref - exact) / np.linalg.norm(exact) < 0.15


@pytest.mark.parametrize("B,G", [(1, 32), (2, 128), (3, 64), (4, 128), (6, 32), (8, 128)])
def test_config2_sweep_cases_full_size(B, G):
    N = K = 8192
    k, s, a, b = datagen.logical_quantized(N, K, B, G, seed=1, name=f"sweep-B{B}-G{G}")
    dk = torch.from_numpy(k).cuda()
    pw = cq.cq_repack(cq.cq_pack_codes(dk, B), torch.from_numpy(s).cuda(), torch.from_numpy(np.ascontiguousarray(a)).cuda(),
                      torch.from_numpy(np.ascontiguousarray(b)).cuda(), B, G, N, K)
    xb = datagen.activations(1, K, seed=1, name="x-sweep")
    y = y_to_numpy(cq.cq_gemm(pw, x_to_device(xb), cq.CQ_MODEL_DTYPE))
    ref = oracle.gemm_model(oracle.pack(k, B), s, a, b, B, G, K, xb)
    check_y(y, ref, f"config 2 B={B} G={G}")


@pytest.mark.parametrize("name,K,N", [("gate_up", 4096, 28672), ("down", 14336, 4096)])
@pytest.mark.parametrize("M", [1, 16])
def test_config3_decode_linears(name, K, N, M):
    B, G = 4, 128
    k, s, a, b = datagen.logical_quantized(N, K, B, G, seed=2, name=name)
    dk = torch.from_numpy(k).cuda()
    pw = cq.cq_repack(cq.cq_pack_codes(dk, B), torch.from_numpy(s).cuda(), torch.from_numpy(np.ascontiguousarray(a)).cuda(),
                      torch.from_numpy(np.ascontiguousarray(b)).cuda(), B, G, N, K)
    xb = datagen.activations(M, K, seed=2)
    y = y_to_numpy(cq.cq_gemm(pw, x_to_device(xb), cq.CQ_MODEL_DTYPE))
    cols = np.sort(datagen.stream(2, "cols-" + name).choice(N, 1024, replace=False))
    ref = sampled_reference(k[cols], s[cols], a[cols], b[cols], B, G, K, xb, cq.CQ_MODEL_DTYPE)
    check_y(y[:, cols], ref, f"config 3 {name} M={M}")


@pytest.mark.parametrize("mode", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
@pytest.mark.parametrize("B", [4, 8])
def test_config4_crossover_shape_m1024(B, mode):
    # qkv 4096 -> 6144, activations with 1 % of columns scaled x20, M = 1024
    K, N, G, M = 4096, 6144, 128, 1024
    k, s, a, b = datagen.logical_quantized(N, K, B, G, seed=3, name="qkv")
    dk = torch.from_numpy(k).cuda()
    pw = cq.cq_repack(cq.cq_pack_codes(dk, B), torch.from_numpy(s).cuda(), torch.from_numpy(np.ascontiguousarray(a)).cuda(),
                      torch.from_numpy(np.ascontiguousarray(b)).cuda(), B, G, N, K)
    xb = datagen.activations(M, K, seed=3, outlier_cols=0.01)
    y = y_to_numpy(cq.cq_gemm(pw, x_to_device(xb), mode))
    g = datagen.stream(3, "sample")
    cols = np.sort(g.choice(N, 256, replace=False))
    rows = np.sort(g.choice(M, 48, replace=False))
    ref = sampled_reference(k[cols], s[cols], a[cols], b[cols], B, G, K, xb, mode, rows=rows)
    check_y(y[np.ix_(rows, cols)], ref, f"config 4 B={B} mode={mode}")


@pytest.mark.parametrize("name,K,N", [("gate_up", 8192, 57344), ("down", 28672, 8192)])
@pytest.mark.parametrize("B", [3, 4])
def test_config5_prefill_gemm(name, K, N, B):
    # M = 4096 tokens, Llama-3-70B MLP shapes, model dtype; drawn on the GPU, sampled rows x channels
    G, M = 128, 4096
    k, s, a, b = datagen.logical_quantized_cuda(N, K, B, G, seed=4)
    pw = cq.cq_repack(cq.cq_pack_codes(k, B), s, a, b, B, G, N, K)
    x = datagen.activations_cuda(M, K, seed=4)
    ws = torch.zeros(cq.cq_workspace_bytes(B, G, M, N, K, 0), dtype=torch.uint8, device="cuda")
    y = cq.cq_gemm(pw, x, cq.CQ_MODEL_DTYPE, ws)
    assert cq.cq_gemm_status(ws) == 0
    g = datagen.stream(4, "sample-" + name)
    cols = np.sort(g.choice(N, 256, replace=False))
    rows = np.sort(g.choice(M, 32, replace=False))
    # tile edges on purpose: first and last channel / token of the matrix and of a 128 / 512 tile
    cols[:4] = [0, 127, 128, N - 1]
    rows[:4] = [0, 511, 512, M - 1]
    cols, rows = np.unique(cols), np.unique(rows)
    ci = torch.from_numpy(cols).cuda()
    xb = x.view(torch.int16).cpu().numpy().view(np.uint16)
    ref = sampled_reference(k[ci].cpu().numpy(), s[ci].cpu().numpy(), a[ci].cpu().numpy(), b[ci].cpu().numpy(),
                            B, G, K, xb, cq.CQ_MODEL_DTYPE, rows=rows)
    got = y[torch.from_numpy(rows).cuda()][:, ci].float().cpu().numpy().astype(np.float64)
    check_y(got, ref, f"config 5 {name} B={B}")
