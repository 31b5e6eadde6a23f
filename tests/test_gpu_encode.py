"""GPU parity of the offline encoder steps against the oracle (Sections 4.1 and 4.3): code assignment
and the candidate search are integer decisions taken in fp64 on both sides and must agree exactly;
scales and losses are floating point and agree to rounding."""
import numpy as np
import pytest
import torch

import datagen
import oracle
import paper_2608_06763_b200 as cq

pytestmark = pytest.mark.gpu

OBJ = {"continuous": cq.CQ_FIT_CONTINUOUS, "joint": cq.CQ_FIT_JOINT}


def dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def fitted(kind, N, K, B, G, seed, objective="continuous"):
    W = datagen.weights(kind, N, K, seed=seed, **({"sigma": 0.02} if kind == "normal" else {"b": 0.015}))
    k, s, a, b = oracle.encode(W, B, G, "fast", objective=objective)
    return W, k, s, a, b


@pytest.mark.parametrize("objective", ["continuous", "joint"])
@pytest.mark.parametrize("B,G", [(1, 64), (2, 32), (3, 64), (4, 128), (5, 64), (6, 32), (8, 128), (4, 512)])
def test_assignment_matches_the_oracle_bit_for_bit(B, G, objective):
    N, K = 6, 1024
    W, k, s, a, b = fitted("laplace", N, K, B, G, seed=200 + B)
    s = (s * np.float32(0.9)).astype(np.float32)      # off the fitted point, so the assignment is not a fixed point
    kg = cq.cq_encode_assign(dev(W), B, G, dev(s), dev(a), dev(b), OBJ[objective]).cpu().numpy()
    fn = oracle.assign_group if objective == "continuous" else oracle.assign_group_joint
    ref = np.empty_like(kg)
    for n in range(N):
        for g in range(K // G):
            ref[n, g * G:(g + 1) * G] = fn(W[n, g * G:(g + 1) * G], B, s[n, g], a[n, g], b[n, g])
    assert np.array_equal(kg, ref)
    assert kg.min() >= -((1 << (B - 1)) - 1) or B == 1      # the reserved pattern is never produced


@pytest.mark.parametrize("objective", ["continuous", "joint"])
@pytest.mark.parametrize("B", [1, 3, 4, 8])
def test_scale_and_losses_match_the_oracle(B, objective):
    N, K, G = 5, 512, 128
    W, k, s, a, b = fitted("normal", N, K, B, G, seed=210 + B, objective=objective)
    sg = cq.cq_encode_scale(dev(W), dev(k), B, G, dev(a), dev(b), OBJ[objective]).cpu().numpy()
    lc, la = cq.cq_encode_losses(dev(W), dev(k), B, G, dev(s), dev(a), dev(b))
    lc, la = lc.cpu().numpy(), la.cpu().numpy()
    for n in range(N):
        for g in range(K // G):
            w, kk = W[n, g * G:(g + 1) * G], k[n, g * G:(g + 1) * G]
            if objective == "joint" or B <= 2:
                want = oracle.joint_scale(w, kk, B, a[n, g], b[n, g])
            else:                                               # continuous analogue: sum u z / sum z^2
                z, _ = oracle.joint_levels(B, a[n, g], b[n, g])
                i = np.abs(kk.astype(np.int64))
                want = float(np.sum(np.abs(w.astype(np.float64)) * z[i]) / np.sum(z[i] ** 2))
            assert sg[n, g] == pytest.approx(want, rel=1e-6)
            rc, ra = oracle.group_losses(w, B, s[n, g], a[n, g], b[n, g], kk)
            assert lc[n, g] == pytest.approx(rc, rel=1e-10, abs=1e-30) and la[n, g] == pytest.approx(ra, rel=1e-10, abs=1e-30)


@pytest.mark.parametrize("objective", ["continuous", "joint"])
@pytest.mark.parametrize("B,G,effort", [(1, 64, "fast"), (2, 64, "fast"), (3, 64, "fast"), (4, 128, "fast"), (4, 32, "int_clipped"),
                                        (6, 64, "fast"), (8, 128, "fast"), (4, 64, "int_absmax"), (3, 32, "reference")])
def test_search_reproduces_the_oracle_encoder(B, G, effort, objective):
    # same candidates, same fp64 decisions: codes and stored parameters are identical; a zero group and an
    # outlier-heavy group ride along
    N, K = 4, 512
    W = datagen.weights("laplace", N, K, seed=220 + B, b=0.015)
    W[1, :G] = 0.0
    W[2, G:2 * G] *= np.where(np.arange(G) % 17 == 0, 12.0, 1.0).astype(np.float32)
    kr, sr, ar, br = oracle.encode(W, B, G, effort, objective=objective)
    kg, sg, ag, bg = cq.cq_encode(dev(W), B, G, OBJ[objective], effort)
    torch.cuda.synchronize()
    assert np.array_equal(kg.cpu().numpy(), kr)
    assert np.array_equal(sg.cpu().numpy(), sr)
    assert np.array_equal(ag.cpu().numpy().view(np.uint16), ar.view(np.uint16))
    assert np.array_equal(bg.cpu().numpy().view(np.uint16), br.view(np.uint16))


def test_encoded_on_the_gpu_runs_through_the_hot_path():
    # encode -> pack -> repack -> GEMV, against the oracle product of the oracle-encoded matrix
    N, K, B, G = 256, 1024, 4, 128
    W = datagen.weights("normal", N, K, seed=230, sigma=0.02)
    k, s, a, b = cq.cq_encode(dev(W), B, G, cq.CQ_FIT_JOINT, "fast")
    pw = cq.cq_repack(cq.cq_pack_codes(k, B), s, a, b, B, G, N, K)
    x = datagen.activations(2, K, seed=231)
    xd = torch.from_numpy(x.view(np.int16)).cuda().view(torch.bfloat16)
    kr, sr, ar, br = oracle.encode(W, B, G, "fast", objective="joint")
    codes = oracle.pack(kr, B)
    for mode in (cq.CQ_MODEL_DTYPE, cq.CQ_DYN_A8):
        y = cq.cq_gemm(pw, xd, mode).float().cpu().numpy().astype(np.float64)
        if mode == cq.CQ_MODEL_DTYPE:
            ref = oracle.gemm_model(codes, sr, ar, br, B, G, K, x)
        else:
            x8, dx = oracle.quantize_a8(x)
            ref = oracle.gemm_a8(codes, sr, ar, br, B, G, K, x8, dx)
        assert np.linalg.norm(y - ref) <= 5e-3 * np.linalg.norm(ref)
