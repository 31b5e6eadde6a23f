"""Routed execution (Section 5.5) through cq_gemm_routed against the oracle: route-major outputs, routes grouped by
matrix, matrices without routes, blocks on both sides of the small-M / large-M dispatch boundary, both modes."""
import ctypes

import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2608_06763_b200 as cq
from util import Case, check_y, y_to_numpy

pytestmark = pytest.mark.gpu


def experts_for(E, N, K, B, G, seed):
    cases, dicts = [], []
    for e in range(E):
        W = datagen.weights("normal", N, K, seed=seed + e, sigma=0.03)
        k, s, a, b = oracle.encode(W, B, G, "fast")
        c = Case(k, s, a, b, B, G)
        cases.append(c)
        dicts.append(dict(codes=c.codes, s=s, a=a, b=b, B=B, G=G, K=K))
    return cases, dicts


@pytest.mark.parametrize("mode", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
@pytest.mark.parametrize("B,G", [(4, 128), (3, 64)])
def test_routed_matches_oracle(B, G, mode):
    E, N, K, T = 5, 200, 512, 64
    cases, dicts = experts_for(E, N, K, B, G, seed=80)
    xb = datagen.activations(T, K, seed=90, outlier_cols=0.01)
    g = datagen.stream(91, "routes")
    counts = [1, 0, 12, 40, 75]                                   # one-token kernel, none, MMA GEMV, tcgen05 with one and two token tiles
    offset = np.concatenate([[0], np.cumsum(counts)])
    route_token = np.concatenate([g.integers(0, T, c) for c in counts]).astype(np.int32)
    y = y_to_numpy(cq.cq_gemm_routed([c.pw for c in cases], torch.from_numpy(xb.view(np.int16)).cuda().view(torch.bfloat16),
                                     torch.from_numpy(route_token).cuda(), offset, mode))
    ref = oracle.gemm_routed(dicts, xb, route_token, offset, "model" if mode == cq.CQ_MODEL_DTYPE else "a8")
    for e in range(E):
        if counts[e]:
            check_y(y[offset[e]:offset[e + 1]], ref[offset[e]:offset[e + 1]], f"routed matrix {e} B={B} mode={mode}")
    # a route is the same bits as the single-matrix call on its gathered rows
    e = 3
    xe = torch.from_numpy(xb[route_token[offset[e]:offset[e + 1]]].view(np.int16)).cuda().view(torch.bfloat16)
    single = y_to_numpy(cq.cq_gemm(cases[e].pw, xe, mode))
    assert np.array_equal(single, y[offset[e]:offset[e + 1]])


def test_routed_argument_errors_and_bad_token():
    E, N, K, T = 2, 128, 256, 4
    cases, dicts = experts_for(E, N, K, 4, 128, seed=95)
    xb = datagen.activations(T, K, seed=96)
    x = torch.from_numpy(xb.view(np.int16)).cuda().view(torch.bfloat16)
    # a token index outside [0, T) reads nothing: its route sees a zero row
    rt = torch.tensor([2, 9, -1], dtype=torch.int32, device="cuda")
    y = y_to_numpy(cq.cq_gemm_routed([c.pw for c in cases], x, rt, [0, 2, 3]))
    assert np.all(y[1] == 0) and np.all(y[2] == 0) and np.any(y[0] != 0)
    L = cq.lib()
    off = (ctypes.c_int64 * 3)(0, 2, 3)
    bad = (ctypes.c_int64 * 3)(0, 3, 2)
    ptrs = (ctypes.c_void_p * 2)(16, 16)
    one = 16
    assert L.cq_gemm_routed(ptrs, 2, 4, 128, one, one, bad, one, 4, 128, 256, 0, 0, one, 1 << 30, None) == -1    # offsets decrease
    assert L.cq_gemm_routed(ptrs, 2, 4, 128, one, one, off, one, 4, 128, 256, 0, 0, one, 64, None) == -4          # workspace
    assert L.cq_gemm_routed(None, 2, 4, 128, one, one, off, one, 4, 128, 256, 0, 0, one, 1 << 30, None) == -1
    assert L.cq_routed_workspace_bytes(4, 128, 2, off, 128, 256, 0) > 0
    assert L.cq_routed_workspace_bytes(4, 128, 2, bad, 128, 256, 0) == 0
