"""Parity at the full sizes of the five benchmark configurations, in the launch configuration the
benchmark times (same entry point, same dispatch, weights produced the same way), on outputs the oracle
computes one by one: whole y where that is cheap, otherwise a seeded sample of activation rows x output
channels that always includes the first and last channel / token of the matrix and of a tile.

Weights follow the configurations' recipes: drawn from the stated distribution and fitted by the
encoder.  Configuration 1 is fitted by the oracle encoder itself; the larger tensors by cq_encode, whose
output is the oracle encoder's bit for bit (tests/test_gpu_encode.py at small sizes, and re-checked here
on sampled rows of every full-size tensor).  The 10^8 .. 10^9-entry tensors of configurations 3 - 5 are
drawn with the seeded GPU generator of datagen.weights_cuda."""
import functools

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


def sample_with_edges(gen, n, count, tile):
    """`count` seeded indices of range(n) plus the first / last index of the range and of a tile."""
    idx = gen.choice(n, min(count, n), replace=False)
    edges = [0, n - 1, tile - 1, tile, n - tile, n // 2]
    return np.unique(np.concatenate([idx, [e for e in edges if 0 <= e < n]]))


class Fitted:
    """A full-size tensor fitted on the GPU, packed for the library, with host copies of sampled channels."""

    def __init__(self, W, B, G, sample_gen, n_cols):
        self.B, self.G = B, G
        self.N, self.K = W.shape
        k, s, a, b = cq.cq_encode(W, B, G, cq.CQ_FIT_CONTINUOUS, "fast")
        self.pw = cq.cq_repack(cq.cq_pack_codes(k, B), s, a, b, B, G, self.N, self.K)
        self.cols = sample_with_edges(sample_gen, self.N, n_cols, 128)
        ci = torch.from_numpy(self.cols).cuda()
        self.k, self.s = k[ci].cpu().numpy(), s[ci].cpu().numpy()
        self.a, self.b = a[ci].cpu().numpy(), b[ci].cpu().numpy()
        # the encoder on the GPU and the oracle encoder agree on these rows bit for bit
        probe = self.cols[:: max(1, len(self.cols) // 6)][:6]
        Wp = W[torch.from_numpy(probe).cuda()].cpu().numpy()
        ko, so, ao, bo = oracle.encode(Wp, B, G, "fast")
        sel = np.searchsorted(self.cols, probe)
        assert np.array_equal(ko, self.k[sel]) and np.array_equal(so, self.s[sel])
        assert np.array_equal(np.asarray(ao).view(np.uint16), self.a[sel].view(np.uint16))
        assert np.array_equal(np.asarray(bo).view(np.uint16), self.b[sel].view(np.uint16))

    def check(self, x, mode, what, rows=None):
        """x: bf16 [M, K] on the device."""
        M = x.shape[0]
        ws = torch.zeros(cq.cq_workspace_bytes(self.B, self.G, M, self.N, self.K, mode), dtype=torch.uint8, device="cuda")
        y = cq.cq_gemm(self.pw, x, mode, ws)
        assert cq.cq_gemm_status(ws) == 0
        xb = x.view(torch.int16).cpu().numpy().view(np.uint16)
        ref = sampled_reference(self.k, self.s, self.a, self.b, self.B, self.G, self.K, xb, mode, rows=rows)
        ci = torch.from_numpy(self.cols).cuda()
        got = y[:, ci] if rows is None else y[torch.from_numpy(rows).cuda()][:, ci]
        check_y(got.float().cpu().numpy().astype(np.float64), ref, what)


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


@functools.lru_cache(maxsize=1)
def sweep_matrix():
    # configuration 2: one 8192 x 8192 Laplace(0, 0.015) matrix, seed 1, for every (B, G) of the sweep
    return torch.from_numpy(datagen.weights("laplace", 8192, 8192, seed=1, b=0.015)).cuda()


@pytest.mark.parametrize("G", [32, 64, 128])
@pytest.mark.parametrize("B", [1, 2, 3, 4, 6, 8])
def test_config2_sweep_all_cases_full_size(B, G):
    f = Fitted(sweep_matrix(), B, G, datagen.stream(1, f"cols-sweep-{B}-{G}"), 1024)
    x = x_to_device(datagen.activations(1, 8192, seed=1, name="x-sweep"))
    f.check(x, cq.CQ_MODEL_DTYPE, f"config 2 B={B} G={G}")


@functools.lru_cache(maxsize=2)
def decode_linear(name, seed):
    # configurations 3 and 4: N(0, 0.02^2) with 0.1 % of the entries replaced by N(0, 0.2^2)
    K, N = {n: (k, nn) for n, k, nn in datagen.LLAMA8B_SHAPES}[name]
    return datagen.weights_cuda("outlier", N, K, seed=seed, sigma=0.02, sigma_out=0.2, p=0.001)


@pytest.mark.parametrize("name", ["qkv", "o", "gate_up", "down"])
def test_config3_decode_linears_all_shapes_and_rows(name):
    W = decode_linear(name, 2)
    f = Fitted(W, 4, 128, datagen.stream(2, "cols-" + name), 1024)
    for M in (1, 4, 8, 16):
        x = x_to_device(datagen.activations(M, W.shape[1], seed=2, name=f"x-{M}"))
        f.check(x, cq.CQ_MODEL_DTYPE, f"config 3 {name} M={M}")


@pytest.mark.parametrize("B", [4, 8])
@pytest.mark.parametrize("name", ["qkv", "o", "gate_up", "down"])
def test_config4_crossover_all_shapes_rows_and_modes(name, B):
    # same four shapes (seed 3), W4 and W8, M in {1, 16, 64, 256, 1024}, activations with 1 % of the
    # columns scaled x20, both activation modes
    W = decode_linear(name, 3)
    K = W.shape[1]
    f = Fitted(W, B, 128, datagen.stream(3, f"cols-{name}-{B}"), 256)
    g = datagen.stream(3, "rows")
    for M in (1, 16, 64, 256, 1024):
        x = datagen.activations_cuda(M, K, seed=3 + M, outlier_cols=0.01)
        rows = None if M <= 64 else sample_with_edges(g, M, 40, 256)
        for mode in (cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8):
            f.check(x, mode, f"config 4 {name} B={B} M={M} mode={mode}", rows=rows)


@pytest.mark.parametrize("name,K,N", [("gate_up", 8192, 57344), ("down", 28672, 8192)])
def test_config5_prefill_gemm_both_modes(name, K, N):
    # M = 4096 tokens, Llama-3-70B MLP shapes, W ~ N(0, 0.015^2) seed 4, W3 and W4, model dtype and Dynamic A8
    M = 4096
    W = datagen.weights_cuda("normal", N, K, seed=4, sigma=0.015)
    x = datagen.activations_cuda(M, K, seed=4)
    g = datagen.stream(4, "sample-" + name)
    rows = sample_with_edges(g, M, 28, 512)
    for B in (3, 4):
        f = Fitted(W, B, 128, g, 200)
        for mode in (cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8):
            f.check(x, mode, f"config 5 {name} B={B} mode={mode}", rows=rows)
        del f
        torch.cuda.empty_cache()
