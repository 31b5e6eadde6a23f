"""Seeded synthetic inputs for the CubicQuant packed GEMV/GEMM path.

This module only draws numbers.  It holds none of the method's arithmetic: no
level function, no bit packing, no quantiser, no encoder.  Both the CPU oracle
and the CUDA library consume what it produces, each with its own code.

Streams are counter based (Philox 4x64 keyed by ``(seed, tensor name)``) and
every transform from raw 64-bit words to a distribution is written out here, so
values do not depend on numpy's distribution routines:

* ``uniform01``   53-bit mantissa uniforms in (0, 1)
* ``normal``      Box-Muller on pairs of uniforms
* ``laplace``     inverse CDF  -b * sgn(u - 1/2) * ln(1 - 2|u - 1/2|)

Workload recipes (the five benchmark configurations) are at the bottom.
"""
from __future__ import annotations

import zlib

import numpy as np

__all__ = [
    "stream", "uniform01", "normal", "laplace", "uniform_pm", "to_bf16_bits",
    "bf16_bits_to_f32", "weights", "activations", "logical_quantized",
    "random_shape_params", "LLAMA8B_SHAPES", "LLAMA70B_MLP_SHAPES",
]


# --------------------------------------------------------------------------- streams
def stream(seed: int, name: str) -> np.random.Generator:
    """Counter-based generator for the tensor called ``name`` under ``seed``."""
    key = np.array([np.uint64(seed), np.uint64(zlib.crc32(name.encode()))], dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def _raw(gen: np.random.Generator, n: int) -> np.ndarray:
    return gen.bit_generator.random_raw(n)


def uniform01(gen: np.random.Generator, n: int) -> np.ndarray:
    """Uniform doubles strictly inside (0, 1): (top 53 bits + 0.5) / 2^53."""
    return ((_raw(gen, n) >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(gen: np.random.Generator, n: int) -> np.ndarray:
    """Standard normal doubles by Box-Muller."""
    h = (n + 1) // 2
    u1 = uniform01(gen, h)
    u2 = uniform01(gen, h)
    r = np.sqrt(-2.0 * np.log(u1))
    th = 2.0 * np.pi * u2
    out = np.empty(2 * h, dtype=np.float64)
    out[0::2] = r * np.cos(th)
    out[1::2] = r * np.sin(th)
    return out[:n]


def laplace(gen: np.random.Generator, n: int, b: float = 1.0) -> np.ndarray:
    """Laplace(0, b) doubles by inverse CDF."""
    d = uniform01(gen, n) - 0.5
    return -b * np.sign(d) * np.log1p(-2.0 * np.abs(d))


def uniform_pm(gen: np.random.Generator, n: int, half_width: float) -> np.ndarray:
    """Uniform doubles on (-half_width, half_width)."""
    return (2.0 * uniform01(gen, n) - 1.0) * half_width


# --------------------------------------------------------------------------- bf16 I/O
def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float -> bfloat16 bit patterns (uint16), round to nearest even."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> the float32 values they denote (exact)."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- tensors
def weights(kind: str, N: int, K: int, seed: int, name: str = "W", **kw) -> np.ndarray:
    """fp32 weight matrix [N, K] (N output channels, K input channels).

    kind = "normal"   : N(0, sigma^2)                                   kw: sigma
           "laplace"  : Laplace(0, b)                                   kw: b
           "outlier"  : N(0, sigma^2), each entry independently replaced
                        with probability p by N(0, sigma_out^2)         kw: sigma, sigma_out, p
           "uniform"  : Uniform(-a, a)                                  kw: a
    """
    g = stream(seed, name)
    n = N * K
    if kind == "normal":
        w = normal(g, n) * kw.get("sigma", 0.02)
    elif kind == "laplace":
        w = laplace(g, n, kw.get("b", 0.015))
    elif kind == "uniform":
        w = uniform_pm(g, n, kw.get("a", 0.05))
    elif kind == "outlier":
        w = normal(g, n) * kw.get("sigma", 0.02)
        sel = uniform01(g, n) < kw.get("p", 0.001)
        big = normal(g, n) * kw.get("sigma_out", 0.2)
        w = np.where(sel, big, w)
    else:
        raise ValueError(kind)
    return w.astype(np.float32).reshape(N, K)


def activations(M: int, K: int, seed: int, name: str = "x", outlier_cols: float = 0.0,
                outlier_scale: float = 20.0) -> np.ndarray:
    """bf16 activation bit patterns [M, K]: N(0,1), optionally with a seeded
    choice of floor(outlier_cols * K) input channels scaled by ``outlier_scale``
    before the bf16 rounding."""
    g = stream(seed, name)
    x = normal(g, M * K).reshape(M, K)
    n_out = int(outlier_cols * K)
    if n_out > 0:
        order = np.argsort(uniform01(stream(seed, name + ".cols"), K), kind="stable")
        x[:, order[:n_out]] *= outlier_scale
    return to_bf16_bits(x)


def random_shape_params(n: int, seed: int, name: str = "params"):
    """Seeded per-group parameters (scale fp32, a fp16, b fp16) as they would
    come out of a fit: a in [0.5, 1], b in [-0.3, 0] (inside the strictly
    monotone domain for every such pair), scale in [0.03, 0.09]."""
    g = stream(seed, name)
    s = (0.03 + 0.06 * uniform01(g, n)).astype(np.float32)
    a = (0.5 + 0.5 * uniform01(g, n)).astype(np.float16)
    b = (-0.3 * uniform01(g, n)).astype(np.float16)
    return s, a, b


def logical_quantized(N: int, K: int, B: int, G: int, seed: int, name: str = "Q"):
    """A seeded, already-quantised tensor in *logical* form, for sizes where
    running a fitter is too slow: signed codes k[N, K] (int8; B=1: +-1, else
    in [-(2^(B-1)-1), 2^(B-1)-1], bell shaped around 0 like fitted codes) and
    per-group (scale, a, b) of shape [N, K/G].  Packing into a byte stream is
    left to the consumer."""
    assert K % G == 0
    g = stream(seed, name)
    n = N * K
    if B == 1:
        k = np.where(uniform01(g, n) < 0.5, -1, 1).astype(np.int8)
    else:
        Mx = (1 << (B - 1)) - 1
        v = laplace(g, n, 0.22 * Mx + 0.35)
        k = np.clip(np.rint(v), -Mx, Mx).astype(np.int8)
    s, a, b = random_shape_params(N * (K // G), seed, name + ".params")
    shp = (N, K // G)
    return k.reshape(N, K), s.reshape(shp), a.reshape(shp), b.reshape(shp)


# --------------------------------------------------------------------------- recipes
# (name, K, N) of the decode linears and the prefill MLP; dimensions only.
LLAMA8B_SHAPES = [("qkv", 4096, 6144), ("o", 4096, 4096),
                  ("gate_up", 4096, 28672), ("down", 14336, 4096)]
LLAMA70B_MLP_SHAPES = [("gate_up", 8192, 57344), ("down", 28672, 8192)]


def logical_quantized_cuda(N: int, K: int, B: int, G: int, seed: int, device="cuda"):
    """Same recipe as ``logical_quantized`` (bell-shaped signed codes, shape parameters in the
    strictly monotone domain, scales in [0.03, 0.09]) drawn with torch's seeded generator on the
    GPU, for tensors too large to draw with numpy in reasonable time.  Returns torch tensors
    (k int8 [N, K], s fp32, a fp16, b fp16 of shape [N, K/G]) on ``device``.  The stream differs
    from the numpy one; consumers that need the values on the CPU copy them back."""
    import torch
    assert K % G == 0
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed) * 1000003 + B * 131 + G)
    k = torch.empty((N, K), dtype=torch.int8, device=device)
    rows = max(1, (1 << 26) // K)  # draw in slabs to bound temporary memory
    for r0 in range(0, N, rows):
        r1 = min(N, r0 + rows)
        u = torch.rand((r1 - r0, K), generator=gen, device=device, dtype=torch.float32)
        if B == 1:
            k[r0:r1] = torch.where(u < 0.5, -1, 1).to(torch.int8)
        else:
            Mx = (1 << (B - 1)) - 1
            d = (u - 0.5).clamp(-0.4999999, 0.4999999)
            v = -(0.22 * Mx + 0.35) * torch.sign(d) * torch.log1p(-2.0 * d.abs())
            k[r0:r1] = v.round().clamp(-Mx, Mx).to(torch.int8)
    n = N * (K // G)
    s = (0.03 + 0.06 * torch.rand(n, generator=gen, device=device)).to(torch.float32).reshape(N, K // G)
    a = (0.5 + 0.5 * torch.rand(n, generator=gen, device=device)).to(torch.float16).reshape(N, K // G)
    b = (-0.3 * torch.rand(n, generator=gen, device=device)).to(torch.float16).reshape(N, K // G)
    return k, s, a, b


def weights_cuda(kind: str, N: int, K: int, seed: int, device="cuda", **kw):
    """fp32 weight matrix [N, K] of the same distributions as ``weights`` (normal / laplace / outlier), drawn
    with torch's seeded generator on the GPU for tensors of 10^8 .. 10^9 entries (the numpy stream takes
    minutes there).  The stream differs from the numpy one."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed) * 2654435761 % (1 << 31) + {"normal": 1, "laplace": 2, "outlier": 3}[kind])
    W = torch.empty((N, K), dtype=torch.float32, device=device)
    rows = max(1, (1 << 25) // K)  # slabs bound the temporaries
    for r0 in range(0, N, rows):
        r1 = min(N, r0 + rows)
        shp = (r1 - r0, K)
        if kind == "normal":
            W[r0:r1] = torch.randn(shp, generator=gen, device=device) * kw.get("sigma", 0.02)
        elif kind == "laplace":
            d = (torch.rand(shp, generator=gen, device=device) - 0.5).clamp(-0.4999999, 0.4999999)
            W[r0:r1] = -kw.get("b", 0.015) * torch.sign(d) * torch.log1p(-2.0 * d.abs())
        elif kind == "outlier":
            base = torch.randn(shp, generator=gen, device=device) * kw.get("sigma", 0.02)
            sel = torch.rand(shp, generator=gen, device=device) < kw.get("p", 0.001)
            big = torch.randn(shp, generator=gen, device=device) * kw.get("sigma_out", 0.2)
            W[r0:r1] = torch.where(sel, big, base)
        else:
            raise ValueError(kind)
    return W


def activations_cuda(M: int, K: int, seed: int, outlier_cols: float = 0.0, outlier_scale: float = 20.0, device="cuda"):
    """bf16 N(0,1) activations [M, K] drawn on the GPU (optionally a seeded set of columns scaled)."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed) * 7919 + 17)
    x = torch.randn((M, K), generator=gen, device=device, dtype=torch.float32)
    n_out = int(outlier_cols * K)
    if n_out > 0:
        cols = torch.randperm(K, generator=gen, device=device)[:n_out]
        x[:, cols] *= outlier_scale
    return x.to(torch.bfloat16)
