"""Helpers shared by the GPU parity tests: build a quantised case with the oracle, move it to the
device through the C ABI, compare."""
import numpy as np
import torch

import datagen
import oracle
import paper_2608_06763_b200 as cq


class Case:
    """Canonical tensors (numpy, from the oracle) and their device copies."""

    def __init__(self, k, s, a, b, B, G):
        self.B, self.G = B, G
        self.N, self.K = k.shape
        self.k, self.s, self.a, self.b = k, s, a, b
        self.codes = oracle.pack(k, B)
        dev = "cuda"
        self.d_codes = torch.from_numpy(self.codes).to(dev)
        self.d_s = torch.from_numpy(np.ascontiguousarray(s)).to(dev)
        self.d_a = torch.from_numpy(np.ascontiguousarray(a).view(np.float16)).to(dev)
        self.d_b = torch.from_numpy(np.ascontiguousarray(b).view(np.float16)).to(dev)
        self.pw = cq.cq_repack(self.d_codes, self.d_s, self.d_a, self.d_b, B, G, self.N, self.K)


def encoded_case(kind, N, K, B, G, seed, effort="fast", **kw):
    W = datagen.weights(kind, N, K, seed=seed, **kw)
    k, s, a, b = oracle.encode(W, B, G, effort)
    return Case(k, s, a, b, B, G)


def logical_case(N, K, B, G, seed):
    k, s, a, b = datagen.logical_quantized(N, K, B, G, seed)
    return Case(k, s, a, b, B, G)


def x_to_device(x_bits):
    return torch.from_numpy(x_bits.view(np.int16)).cuda().view(torch.bfloat16)


def y_to_numpy(y):
    return y.float().cpu().numpy().astype(np.float64)


def rel_fro(y, ref):
    return float(np.linalg.norm(y - ref) / max(np.linalg.norm(ref), 1e-300))


def check_y(y, ref, what=""):
    """spec tolerance: relative Frobenius <= 5e-3 and max |y - ref| <= 1e-2 max|ref|."""
    fro = rel_fro(y, ref)
    mx = float(np.abs(y - ref).max() / max(np.abs(ref).max(), 1e-300))
    assert fro <= 5e-3 and mx <= 1e-2, f"{what}: rel_fro={fro:.3e} max_rel={mx:.3e}"
    return fro, mx
