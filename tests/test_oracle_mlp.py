"""Pins of the oracle's fused-MLP composition (Section 5.4, last paragraph)."""
import numpy as np

import datagen
import oracle


def part(W, B, G):
    k, s, a, b = oracle.encode(W, B, G, "fast")
    return dict(codes=oracle.pack(k, B), s=s, a=a, b=b, B=B, G=G, K=W.shape[1], k=k)


def test_gated_activation_identities():
    g = np.linspace(-30, 30, 2001)
    u = np.cos(g) + 1.5
    act = oracle.silu_mul(g, u)
    assert np.all(oracle.silu_mul(np.zeros(5), np.arange(5.0)) == 0.0)                       # silu(0) = 0
    assert np.allclose(act - oracle.silu_mul(-g, u), g * u, rtol=1e-14, atol=1e-14)          # silu(g) - silu(-g) = g
    big = g > 25
    assert np.allclose(act[big], (g * u)[big], rtol=1e-10)                                   # silu(g) -> g
    assert np.allclose(oracle.silu_mul(1.0, 1.0), 1.0 / (1.0 + np.exp(-1.0)), rtol=1e-15)    # the logistic value at 1
    assert np.all(np.diff(oracle.silu_mul(g[g > -1.27], 1.0)) > 0)                           # increasing right of its minimum


def test_mlp_composition_special_cases():
    K, I, N, M = 256, 128, 64, 5
    Wgu = datagen.weights("normal", 2 * I, K, seed=31)
    Wdn = datagen.weights("normal", N, I, seed=32)
    x = datagen.activations(M, K, seed=33)
    gu, dn = part(Wgu, 4, 64), part(Wdn, 4, 64)
    y, act = oracle.mlp_swiglu(gu, dn, x)
    assert y.shape == (M, N) and act.shape == (M, I)
    # the down projection sees exactly the quantised activation: redo its product from act by the A8 oracle
    a8, da = oracle.quantize_a8(act)
    assert np.array_equal(y, oracle.gemm_a8(dn["codes"], dn["s"], dn["a"], dn["b"], 4, 64, I, a8, da))
    # a zero gate gives a zero activation and a zero output whatever the up half holds
    kz = gu["k"].copy()
    kz[:I] = 0
    gz = dict(gu, codes=oracle.pack(kz, 4))
    yz, az = oracle.mlp_swiglu(gz, dn, x)
    assert np.all(datagen.bf16_bits_to_f32(az) == 0.0) and np.all(yz == 0.0)
    # against the unquantised chain: two 4-bit projections and an INT8 activation stay within a loose bound
    xf = datagen.bf16_bits_to_f32(x).astype(np.float64)
    h = xf @ Wgu.astype(np.float64).T
    exact = oracle.silu_mul(h[:, :I], h[:, I:]) @ Wdn.astype(np.float64).T
    assert np.linalg.norm(y - exact) / np.linalg.norm(exact) < 0.35
    # both gate_up modes agree to within the A8 error of one projection
    y8, _ = oracle.mlp_swiglu(gu, dn, x, mode_gate_up="a8")
    assert np.linalg.norm(y8 - y) / np.linalg.norm(y) < 0.05
