"""The fused MLP boundary (Section 5.4, last paragraph) against the oracle's composition of the operators it
fuses, and against the same chain run operator by operator on the GPU."""
import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2608_06763_b200 as cq
from util import Case, rel_fro, x_to_device, y_to_numpy

pytestmark = pytest.mark.gpu


def fitted(N, K, B, G, seed):
    W = datagen.weights("normal", N, K, seed=seed, sigma=0.03)
    k, s, a, b = oracle.encode(W, B, G, "fast")
    c = Case(k, s, a, b, B, G)
    return c, dict(codes=c.codes, s=s, a=a, b=b, B=B, G=G, K=K)


@pytest.mark.parametrize("mode_gu", [cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8])
@pytest.mark.parametrize("M", [1, 8, 16, 40, 300])
@pytest.mark.parametrize("Bgu,Ggu,Bdn,Gdn", [(4, 128, 4, 128), (3, 64, 8, 32)])
def test_fused_mlp_matches_the_oracle_chain(Bgu, Ggu, Bdn, Gdn, M, mode_gu):
    K, I, N = 512, 384, 200
    cgu, ogu = fitted(2 * I, K, Bgu, Ggu, seed=40)
    cdn, odn = fitted(N, I, Bdn, Gdn, seed=41)
    xb = datagen.activations(M, K, seed=42 + M, outlier_cols=0.01)
    x = x_to_device(xb)
    need = cq.lib().cq_mlp_workspace_bytes(Bgu, Ggu, Bdn, Gdn, M, K, I, N, mode_gu)
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    y = y_to_numpy(cq.cq_mlp_swiglu(cgu.pw, cdn.pw, x, mode_gu, ws))
    assert cq.cq_gemm_status(ws) == 0
    ref, _ = oracle.mlp_swiglu(ogu, odn, xb, "model" if mode_gu == cq.CQ_MODEL_DTYPE else "a8")
    # Tolerance of the chain: the first operator is within 5e-3 of its oracle, so the two chains quantise slightly
    # different activations; a deviation of that size moves roughly a tenth of them across an INT8 rounding boundary,
    # i.e. by a whole step of max|act| / 127, which is noise of the order of the A8 quantisation error itself
    # (about 1 % of y).  The chain is therefore held to 2e-2 relative Frobenius and 3e-2 of the largest output.
    fro = rel_fro(y, ref)
    mx = np.abs(y - ref).max() / np.abs(ref).max()
    assert fro <= 2e-2 and mx <= 3e-2, (fro, mx)
    # the same chain operator by operator on the GPU: gate_up, an elementwise activation in fp32, down in Dynamic A8;
    # the fused kernel may only differ where its fp32 activation rounds to the neighbouring bf16 value
    h = cq.cq_gemm(cgu.pw, x, mode_gu).float()
    act = (torch.nn.functional.silu(h[:, :I]) * h[:, I:]).to(torch.bfloat16)
    y2 = y_to_numpy(cq.cq_gemm(cdn.pw, act, cq.CQ_DYN_A8))
    assert rel_fro(y, y2) <= 2.5e-3, rel_fro(y, y2)
    # a second call on the same workspace reproduces the first bit for bit
    y3 = y_to_numpy(cq.cq_mlp_swiglu(cgu.pw, cdn.pw, x, mode_gu, ws))
    assert np.array_equal(y, y3)


def test_fused_mlp_f16_and_argument_errors():
    K, I, N, M = 256, 256, 128, 5
    cgu, ogu = fitted(2 * I, K, 4, 128, seed=50)
    cdn, odn = fitted(N, I, 4, 128, seed=51)
    xh = datagen.bf16_bits_to_f32(datagen.activations(M, K, seed=52)).astype(np.float16)
    y = cq.cq_mlp_swiglu(cgu.pw, cdn.pw, torch.from_numpy(xh).cuda())
    assert y.dtype == torch.float16 and torch.isfinite(y).all()
    # binary16 values that bf16 also holds exactly would give the bf16 chain; here only closeness to it is asked
    yb = cq.cq_mlp_swiglu(cgu.pw, cdn.pw, torch.from_numpy(xh).cuda().to(torch.bfloat16))
    assert rel_fro(y.float().cpu().numpy(), yb.float().cpu().numpy()) < 2e-2
    L = cq.lib()
    one = 16
    assert L.cq_mlp_swiglu(None, 4, 128, one, 4, 128, one, one, 1, 256, 256, 128, 0, 0, one, 1 << 30, None) == -1
    assert L.cq_mlp_swiglu(one, 4, 128, one, 4, 128, one, one, 1, 256, 256, 128, 3, 0, one, 1 << 30, None) == -1   # unknown mode
    assert L.cq_mlp_swiglu(one, 4, 128, one, 4, 128, one, one, 1, 256, 200, 128, 0, 0, one, 1 << 30, None) == -2   # I % G != 0
    assert L.cq_mlp_swiglu(one, 4, 128, one, 4, 128, one, one, 1, 256, 256, 128, 0, 0, one, 64, None) == -4         # workspace
    assert L.cq_mlp_workspace_bytes(4, 128, 4, 128, 1, 256, 256, 128, 0) > 0
