"""Pin of the oracle's routed product (Section 5.5): every route is the ordinary product of its token with its matrix."""
import numpy as np

import datagen
import oracle


def test_routed_equals_route_by_route_dense_products():
    K, N, E, T = 128, 24, 3, 6
    experts, dense = [], []
    for e in range(E):
        W = datagen.weights("normal", N, K, seed=60 + e)
        k, s, a, b = oracle.encode(W, 4, 32, "fast")
        codes = oracle.pack(k, 4)
        experts.append(dict(codes=codes, s=s, a=a, b=b, B=4, G=32, K=K))
        dense.append(oracle.decode_dense(codes, s, a, b, 4, 32, K))
    x = datagen.activations(T, K, seed=70)
    route_token = np.array([4, 0, 5, 1, 1, 3, 2], np.int32)      # matrix 0: routes 0-2, matrix 1: none, matrix 2: routes 3-6
    offset = [0, 3, 3, 7]
    y = oracle.gemm_routed(experts, x, route_token, offset)
    xf = datagen.bf16_bits_to_f32(x).astype(np.float64)
    for r, t in enumerate(route_token):
        e = 0 if r < 3 else 2
        assert np.allclose(y[r], xf[t] @ dense[e].T, rtol=1e-12, atol=1e-15), r
    # Dynamic A8: each route quantises its own token row, exactly as the single-matrix operator does
    y8 = oracle.gemm_routed(experts, x, route_token, offset, mode="a8")
    x8, dx = oracle.quantize_a8(x)
    for r, t in enumerate(route_token):
        e = experts[0 if r < 3 else 2]
        one = oracle.gemm_a8(e["codes"], e["s"], e["a"], e["b"], 4, 32, K, x8[t:t + 1], dx[t:t + 1])
        assert np.array_equal(y8[r:r + 1], one)
